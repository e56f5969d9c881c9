/*
 * compams.h - C ABI of the B200 (sm_100a) COMP-AMS optimizer-step library.
 *
 * The library runs ONE iteration of Algorithm 2 ("Distributed COMP-AMS with error feedback") of
 * "On Distributed Adaptive Optimization with Gradient Compression" (Li, Karimi, Li, ICLR 2022)
 * per call, with all n workers held as rows of [n, d] buffers on one GPU:
 *
 *   worker i (Algorithm 2, the corrected-gradient and residual steps):   x_i = g_i + e_i;  g~_i = C(x_i);  e_i <- x_i - g~_i
 *   server   (Algorithm 2, the server's average and update): gbar = (1/n) sum_i g~_i;
 *                                        m <- b1 m + (1-b1) gbar;  v <- b2 v + (1-b2) gbar^2;
 *                                        vhat <- max(vhat, v);  theta <- theta - lr m / sqrt(vhat + eps)
 *
 * C is Top-k (Definition 1) or Block-Sign (Definition 2), applied block by block, the blocks
 * being a contiguous partition of [0, d) (Section 3.1: usually one block per network layer).
 *
 * Conventions
 *   - "host" / "device" after a pointer says where the memory lives. No call takes ownership of
 *     caller memory. All device work is enqueued on the handle's CUDA stream (default: the legacy
 *     default stream); calls return without synchronising unless stated otherwise.
 *   - Every call returns COMPAMS_OK (0) or a negative compams_status. Nothing aborts, throws or
 *     prints. One handle may be used by one host thread at a time, and every call that enqueues work
 *     on a handle must be made with the CUDA device current on which the handle was created
 *     (otherwise: INVALID_ARG, nothing is enqueued).
 *   - All state is fp32. Every fp32 operation of the update is a separately rounded IEEE
 *     operation (no fused multiply-add, IEEE sqrt and division, subnormals kept).
 *   - Gradients must be finite. NaN/Inf make the Top-k selection undefined (no fault, but the
 *     kept set is unspecified).
 */
#ifndef COMPAMS_H
#define COMPAMS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct compams_context* compams_handle;

/* Compressors (Section 3.1). */
enum compams_compressor {
    COMPAMS_TOPK = 0,      /* Definition 1, per block; k_b = clamp(floor(k_ratio * d_b), 1, d_b) */
    COMPAMS_BLOCKSIGN = 1, /* Definition 2: sign(x_B) * ||x_B||_1 / d_B */
    COMPAMS_RANDK = 2      /* Random-k (Section 2.1 lists it beside Top-k): per block, k_b coordinates drawn uniformly
                              at random whatever their values; see compams_set_seed for the drawing rule */
};

enum compams_status {
    COMPAMS_OK = 0,
    COMPAMS_ERR_INVALID_ARG = -1,   /* a null pointer, a size out of range, malformed block offsets ... */
    COMPAMS_ERR_ALLOC = -2,         /* host or device allocation failed */
    COMPAMS_ERR_CUDA = -3,          /* a CUDA runtime call failed (see compams_last_cuda_error) */
    COMPAMS_ERR_DEVICE_STATUS = -4, /* a kernel recorded an internal inconsistency in the status word */
    COMPAMS_ERR_TOO_LARGE = -5      /* the problem exceeds a fixed capacity (compams_blocksign_sweep_static) */
};

/* Buffers readable through compams_get_buffer. */
enum compams_buffer {
    COMPAMS_BUF_E = 0,            /* float  [n, d]   error accumulators e_{t+1,i} (Algorithm 2, the residual update); not
                                                    stored (count 0) when every k_b = d_b: they are identically zero */
    COMPAMS_BUF_M = 1,            /* float  [d]      first moment m_t                                            */
    COMPAMS_BUF_V = 2,            /* float  [d]      second moment v_t                                           */
    COMPAMS_BUF_VHAT = 3,         /* float  [d]      running maximum vhat_t                                      */
    COMPAMS_BUF_GBAR = 4,         /* float  [d]      averaged compressed gradient gbar_t                         */
    COMPAMS_BUF_TOPK_IDX = 5,     /* int32  [n, K]   kept coordinates (index into [0, d)); K = sum_b k_b         */
    COMPAMS_BUF_TOPK_VAL = 6,     /* float  [n, K]   kept values, bit-identical to x at that coordinate          */
    COMPAMS_BUF_TOPK_SEG_OFFSETS = 7, /* int64 [M+1] block b of worker i owns entries [i*K+off[b], i*K+off[b+1]) */
    COMPAMS_BUF_SIGN_BITS = 8,    /* uint32 [n, W]   Block-Sign sign bits, see below; W = sum_b ceil(d_b / 32)   */
    COMPAMS_BUF_SIGN_WORD_OFFSETS = 9, /* int64 [M+1] first word of block b inside a row of SIGN_BITS            */
    COMPAMS_BUF_SCALES = 10,      /* float  [n, M]   Block-Sign scales ||x_B||_1 / d_B                           */
    COMPAMS_BUF_STATUS = 11       /* uint32 [8]      [0] status word (0 = clean); Top-k counters since creation:
                                                    [1] (worker, block) selections done by the dense passes,
                                                    [2] selections done inside the candidate list; why a list
                                                    was given up: [3] fewer candidates than k_b, [4] more than
                                                    its capacity, [5] threshold beyond the histogram's range,
                                                    [6] too many candidates sharing the threshold bin; [7] unused */
};

/* Kernel identifiers for compams_get_kernel_time. */
enum compams_kernel {
    COMPAMS_K_DENSE_MEAN_AMSGRAD = 0, /* k = d: mean over workers fused with the AMSGrad update              */
    COMPAMS_K_BS_SWEEP = 1,           /* Block-Sign: EF add, per-tile |x| sums, sign pack                      */
    COMPAMS_K_BS_APPLY = 2,           /* Block-Sign: segmented average over workers fused with AMSGrad        */
    COMPAMS_K_BS_MATERIALIZE = 3,     /* Block-Sign: turn the stored x into e when E is read                  */
    COMPAMS_K_TOPK_SWEEP = 4,         /* Top-k: EF add, x written to E, candidates above the predicted threshold */
    COMPAMS_K_TOPK_DENSE = 5,         /* Top-k dense passes (one cooperative launch): radix histograms over x,
                                         threshold search, emission, lowest-index ties                        */
    COMPAMS_K_TOPK_MATERIALIZE = 6,   /* Top-k: zero e at the coordinates kept in the last step when E is read   */
    COMPAMS_K_RANDK_EMIT = 7,         /* Random-k: every message slot computes its drawn coordinate and fetches x there */
    /* 8: reserved (never returned, never timed) */
    COMPAMS_K_TOPK_SCATTER = 9,       /* Top-k: closes the step per segment; sparse scatter-accumulate         */
    COMPAMS_K_AMSGRAD = 10,           /* Top-k: AMSGrad update from the accumulated average                   */
    COMPAMS_K_TOPK_SMALL = 11,        /* Top-k: whole small blocks selected inside shared memory              */
    COMPAMS_K_TOPK_SELECT = 12,       /* Top-k: exact selection inside the candidate lists                    */
    COMPAMS_K_BS_SCALES = 13,         /* Block-Sign: scale of every (worker, block) from the tile sums        */
    COMPAMS_K_COUNT = 14
};

/*
 * compams_create - build the optimizer state (Algorithm 2, "Initialize": e_{1,i} = 0,
 * m_0 = v_0 = vhat_0 = 0).
 *
 *   out            host; receives the handle. Untouched on failure.
 *   n              number of simulated workers, 1 <= n <= 65535.
 *   d              number of parameters, 1 <= d <= 2^31 - 32768.
 *   block_offsets  host; num_blocks + 1 entries, [0] = 0, strictly increasing, last = d. Copied.
 *   num_blocks     M >= 1. The compressor acts on each block separately (Section 3.1). With one
 *                  block Top-k is taken over the whole vector; with one block per tensor it is
 *                  layer-wise.
 *   compressor     COMPAMS_TOPK, COMPAMS_BLOCKSIGN or COMPAMS_RANDK.
 *   k_ratio        Top-k and Random-k, in (0, 1]: block b keeps k_b = max(1, min(d_b, floor(k_ratio * d_b)))
 *                  coordinates (Section 5.1 uses 0.01). If every k_b equals d_b the compressor is
 *                  the identity (q = 0 in Assumption 1): the step is then full-precision
 *                  distributed AMSGrad, e stays 0 and no (index, value) message is produced.
 *                  Ignored for Block-Sign.
 *   lr, beta1, beta2, eps   AMSGrad hyper-parameters (Algorithm 1); eps is added under the root.
 *
 * Allocates, on the current CUDA device, E [n, d], m, v, vhat, gbar [d], the message buffers and
 * scratch, all owned by the handle and zero-initialised. Synchronises the device once.
 * Errors: INVALID_ARG for any violated range above; ALLOC; CUDA.
 */
int compams_create(compams_handle* out, int32_t n, int64_t d, const int64_t* block_offsets, int32_t num_blocks,
                   int32_t compressor, double k_ratio, float lr, float beta1, float beta2, float eps);

/*
 * compams_step - one iteration of Algorithm 2 (the corrected-gradient and residual steps for every worker, the server's average and update for the
 * server), enqueued on the handle's stream.
 *
 *   grads   device; [n, d] fp32, packed row-major (row i = g_{t,i}, row stride d), 4-byte aligned.
 *           Read only; must stay valid and unchanged until the enqueued work has run.
 *   theta   device; [d] fp32 parameters theta_t, overwritten with theta_{t+1}. 16-byte aligned.
 *
 * After the step: BUF_E holds e_{t+1}, BUF_GBAR holds gbar_t (while compams_record_average is on),
 * BUF_M/V/VHAT the moments, and
 * the message buffers hold what each worker would have sent: for Top-k the k_b (index, value)
 * pairs of every (worker, block) - in no particular order inside a segment, ties at the
 * threshold magnitude resolved towards the lower index - and for Block-Sign one sign bit per
 * coordinate plus one scale per (worker, block). sign(x) follows the IEEE sign bit (+0 -> +,
 * -0 -> -), so every coordinate of a block contributes exactly +-scale.
 * Errors: INVALID_ARG (null or misaligned pointer), CUDA (launch failure).
 *
 * A step enqueues kernels only (no allocation, no host synchronisation), so it may be captured into a CUDA
 * graph on the handle's stream. What the captured launches bake in are the handle's host-side switches of
 * that moment (which of two alternating buffers is current, whether E still holds the last step's x): they
 * repeat with period two once one step has run, so capture an even number of steps after a first eager
 * step, and refill the captured gradient buffers before every replay. Not for COMPAMS_RANDK (the iteration
 * index that keys its index sets is a kernel argument); compams_bits_transmitted counts captured steps once.
 */
int compams_step(compams_handle h, const float* grads, float* theta);

/*
 * compams_step_bf16 / compams_compress_bf16 - compams_step / compams_compress for gradients stored as
 * bfloat16 (what a mixed-precision backward pass produces): the worker-side read of g shrinks from 4 to
 * 2 bytes per element, everything else is unchanged. The corrected-gradient step of Algorithm 2 becomes x = widen(g) + e with
 * widen exact, so the step equals compams_step on the fp32 tensor that holds the same values, bit for bit;
 * e, the messages and the server state stay fp32. A handle may be fed fp32 in one step and bfloat16 in
 * the next.
 *
 *   grads_bf16   device; [n, d] bfloat16 (16-bit patterns: sign, 8 exponent bits, 7 fraction bits), packed
 *                row-major, 2-byte aligned; read only.
 */
int compams_step_bf16(compams_handle h, const void* grads_bf16, float* theta);
int compams_compress_bf16(compams_handle h, const void* grads_bf16);

/*
 * compams_step_host - the same iteration for callers whose tensors live in HOST memory
 * (the two ends of Algorithm 2's exchange with the server, on a machine where the
 * gradients are produced off-GPU).
 *
 *   grads_host  host; [n, d] fp32 packed. Copied to a device staging buffer owned by the handle.
 *   theta_host  host; [d] fp32; copied in, updated, copied back.
 *
 * Enqueues copy-in, the step and copy-out on the handle's stream and then SYNCHRONISES the
 * stream, so on return theta_host holds theta_{t+1}. Pinned host memory makes the copies faster
 * but is not required. The staging buffers are allocated on first use.
 */
int compams_step_host(compams_handle h, const float* grads_host, float* theta_host);

/*
 * Workers sharded over several handles (several GPUs or processes), as in Algorithm 2 proper: every
 * worker compresses locally and ships its compressed gradient to the server; the server averages
 * the n compressed gradients and updates theta (the server's part). Here every shard also plays the server
 * on its own replica of theta, m, v, vhat: after the shards have exchanged their compressed gradients
 * (an all-gather of the message buffers - the only communication, and it is the caller's: this library
 * starts no collective), each applies the identical update, so the replicas stay bit-identical and
 * theta needs no broadcast. (The update is a function of the gathered messages alone. The one place where
 * the order of arrival could show is the binary64 sum over workers at a coordinate, which is exact - hence
 * order-free - while the magnitudes met at one coordinate lie within about 2^24 of one another at n = 32;
 * beyond that spread the last bit of gbar may differ between replicas, and a job that must exclude even
 * that re-broadcasts theta from one rank now and then.)
 *
 * compams_create_sharded - like compams_create, for a handle that holds workers first_worker ...
 *   first_worker + n_local - 1 of n_total (1 <= n_local, first_worker >= 0,
 *   first_worker + n_local <= n_total <= 65535). E is [n_local, d]; the message buffers
 *   (BUF_TOPK_IDX / BUF_TOPK_VAL [n_total, K], or BUF_SIGN_BITS [n_total, W] and BUF_SCALES
 *   [n_total, M]) have one row per worker of the whole job. The uncompressed mode (every k_b = d_b)
 *   has no message to exchange and is refused (INVALID_ARG). compams_create(n, ...) is
 *   compams_create_sharded(n, n, 0, ...).
 *
 * compams_compress - the workers' loop for this handle's workers: x = g + e, the compression, the residual.
 *   grads   device; [n_local, d] fp32 packed, 4-byte aligned; read only.
 *   Fills rows first_worker ... first_worker + n_local - 1 of the message buffers. The caller then
 *   makes the other rows hold the other shards' messages (for Block-Sign BUF_SCALES must be asked for
 *   AFTER this call: two scale buffers alternate), ordered on the handle's stream before compams_apply.
 *
 * compams_apply - the server's part: gbar_t = (1/n_total) sum of the n_total messages, then the AMSGrad update.
 *   theta   device; [d] fp32, 16-byte aligned; updated in place.
 *
 * compams_step on a handle with n_local == n_total is compams_compress followed by compams_apply;
 * on a sharded handle it returns INVALID_ARG (the exchange is missing). Both calls enqueue on the
 * handle's stream and return without synchronising.
 *
 * Order of calls: compams_compress opens an iteration and compams_apply closes it. In between the
 * residual update of the workers is not yet final, so compams_compress, compams_step, compams_step_host,
 * compams_get_state, compams_set_state and compams_get_buffer(BUF_E) return INVALID_ARG (the message
 * buffers and the server's buffers stay readable); compams_apply without an open iteration returns
 * INVALID_ARG too.
 */
int compams_create_sharded(compams_handle* out, int32_t n_local, int32_t n_total, int32_t first_worker, int64_t d,
                           const int64_t* block_offsets, int32_t num_blocks, int32_t compressor, double k_ratio, float lr,
                           float beta1, float beta2, float eps);
int compams_compress(compams_handle h, const float* grads);
int compams_apply(compams_handle h, float* theta);

/*
 * The handle's state in memory the caller allocates (for a harness that wants every device byte to come from
 * its own allocator, e.g. one torch tensor): Algorithm 2's e, m, v, vhat, the message buffers and all scratch
 * are cut from one region instead of being allocated one by one.
 *
 * compams_workspace_bytes - the size of that region for a handle with the given shape (the arguments mean
 *   what they mean for compams_create_sharded; n_local == n_total for an unsharded handle). Host arithmetic
 *   only: no CUDA call is made, no device is needed.
 *   bytes   host; receives the size, a multiple of 256.
 *
 * compams_create_in_workspace - compams_create_sharded with the state placed in `workspace`.
 *   workspace        device; at least workspace_bytes bytes, 256-byte aligned, on the current device. The caller
 *                    keeps ownership: it must outlive the handle and is not freed by compams_destroy; its
 *                    contents are the handle's while the handle lives.
 *   workspace_bytes  its size; INVALID_ARG when smaller than compams_workspace_bytes reports.
 *   No cudaMalloc is made for the state (small host-side objects - events for per-kernel timing - are still
 *   created on demand, and compams_step_host allocates its staging buffers on first use).
 */
int compams_workspace_bytes(size_t* bytes, int32_t n_local, int32_t n_total, int64_t d, const int64_t* block_offsets,
                            int32_t num_blocks, int32_t compressor, double k_ratio);
int compams_create_in_workspace(compams_handle* out, void* workspace, size_t workspace_bytes, int32_t n_local,
                                int32_t n_total, int32_t first_worker, int64_t d, const int64_t* block_offsets,
                                int32_t num_blocks, int32_t compressor, double k_ratio, float lr, float beta1, float beta2,
                                float eps);

/* compams_destroy - free everything the handle owns (synchronises its stream first).
 * A null handle is a no-op. */
int compams_destroy(compams_handle h);

/* compams_set_stream - use `cuda_stream` (a cudaStream_t passed as void*, null = default stream)
 * for all later work of this handle. The caller orders earlier work against the new stream. */
int compams_set_stream(compams_handle h, void* cuda_stream);

/*
 * compams_set_seed - Random-k: the seed of the index sets and the number of iterations already done (the
 * next step is iteration iterations_done + 1; a new handle starts at seed 0, iterations_done 0; a run resumed
 * from compams_set_state passes the iteration count of the checkpoint). Other compressors ignore both.
 *
 * The drawing rule (Section 2.1 only names Random-k; this is the library's reading, fixed so that a
 * second implementation can reproduce the sets bit for bit): worker i keeps in block b, at iteration t,
 * the coordinates block_offsets[b] + pi(r), r = 0 .. k_b - 1, where pi is a permutation of {0 .. d_b - 1}:
 * a balanced Feistel network of six rounds over the smallest even number of bits 2w with 2^(2w) >= d_b
 * (at least 2), applied again while the result is >= d_b. Round r maps (L, R) to
 * (R, L xor (F(R xor key_r) & (2^w - 1))): F is the 32-bit finalizer of MurmurHash3 (h ^= h >> 16;
 * h *= 0x85ebca6b; h ^= h >> 13; h *= 0xc2b2ae35; h ^= h >> 16) and key_0 .. key_5 are the low and high
 * 32-bit halves of the first three output words of Philox4x64-10 (Salmon et al., SC 2011) at counter
 * (0, 0, b, i) under key (seed, t); the input is L = r >> w, R = r & (2^w - 1), the output (L << w) | R. Workers are numbered
 * over the whole job (first_worker + local index on a sharded handle).
 */
int compams_set_seed(compams_handle h, uint64_t seed, uint64_t iterations_done);

/*
 * compams_record_average - whether the server's update also stores the averaged compressed gradient gbar_t
 * (Algorithm 2, the server's average), readable as COMPAMS_BUF_GBAR. gbar_t is an intermediate: theta, m, v and
 * v-hat are computed from it in registers and nothing later reads it, so a new handle does not store it and the
 * update moves 4 bytes per coordinate less. on != 0: stored from the next compams_step / compams_apply on;
 * 0: not stored, and compams_get_buffer refuses COMPAMS_BUF_GBAR with INVALID_ARG. Every other result is
 * bit-identical in both settings. A step captured in a CUDA graph keeps the setting it was captured with.
 */
int compams_record_average(compams_handle h, int on);

/* compams_set_lr - learning rate eta_t for the following steps (Algorithm 2 allows it to vary
 * with t; Section 5.2 divides it by 10 at fixed epochs). */
int compams_set_lr(compams_handle h, float lr);

/*
 * compams_get_state / compams_set_state - checkpoint and restore what Algorithm 2 carries from one
 * iteration to the next: the workers' error accumulators e_{t,i} (the residual update) and the server's m_t, v_t,
 * v-hat_t (the moment and maximum updates). theta is the caller's own tensor and the step counter does not enter the
 * update (Algorithm 1 has no bias correction), so these four are the whole state.
 *
 *   e         DEVICE, [n, d] packed rows, or null to skip. With k_b = d_b in every block the
 *             accumulators are identically zero and not stored: get writes zeros, set ignores e.
 *   m, v, vhat  DEVICE, [d] each, or null to skip.
 *
 * get copies out the values the residual update defines (a residual still to be finished is finished first);
 * set copies in and forgets what the library had derived from earlier steps (threshold
 * predictions), which changes the path a selection takes, never its result. Both run on the
 * handle's stream, asynchronously; the caller's buffers must stay valid until that work is done.
 * A run continued from a restored state is bit-identical to the uninterrupted one.
 */
int compams_get_state(compams_handle h, float* e, float* m, float* v, float* vhat);
int compams_set_state(compams_handle h, const float* e, const float* m, const float* v, const float* vhat);

/*
 * compams_bits_transmitted - worker-to-server traffic of all steps so far, in bits, under the
 * accounting of Section 5.2 ("Communication Efficiency": 32 bits per floating-point number).
 *
 *   out   host, uint64[3]:
 *         [0] what full-precision gradients would have cost: 32 n d per step;
 *         [1] the compressed payload: per worker and step 32 bits per kept value (Top-k), or one
 *             bit per coordinate plus 32 bits per block scale (Block-Sign); equal to [0] when
 *             every block keeps all its coordinates;
 *         [2] the 32-bit coordinate indices that accompany Top-k values (0 otherwise). The
 *             roughly hundredfold saving the paper reports for Top-0.01 is [0] / [1]; a wire format also pays [2].
 */
int compams_bits_transmitted(compams_handle h, uint64_t* out);

/*
 * compams_get_buffer - device pointer and element count of one of the handle's buffers.
 *
 *   which     a compams_buffer value.
 *   dev_ptr   host; receives the DEVICE pointer (read-only for the caller).
 *   count     host; receives the number of elements (0 if the buffer does not exist for this
 *             compressor, in which case *dev_ptr is null).
 *
 * The contents are those of the last enqueued step once the stream has reached that point;
 * they stay valid until the next compams_step / compams_destroy. Asking for BUF_E enqueues
 * one extra kernel that finishes the residual update of Algorithm 2 in place: the step itself leaves the
 * corrected gradient x in E (Block-Sign: all of it; Top-k: at the kept coordinates, which are the
 * ones whose magnitude reaches a value the selection leaves per worker and block) and applies
 * e = x - g~ when E is next read, by the next iteration's sweep or by this call; the values are
 * identical either way. (Random-k zeroes its kept coordinates at once.)
 *
 * SIGN_BITS layout: row i has W words; block b starts at word SIGN_WORD_OFFSETS[b]; bit (r % 32)
 * of word SIGN_WORD_OFFSETS[b] + r / 32 is the sign bit of x at coordinate block_offsets[b] + r;
 * unused high bits of a block's last word are 0.
 */
int compams_get_buffer(compams_handle h, int32_t which, void** dev_ptr, int64_t* count);

/* compams_check_status - synchronise the handle's stream, read the device status word and any
 * pending CUDA error. Returns OK, ERR_CUDA or ERR_DEVICE_STATUS; *status_word (host, may be null)
 * receives the raw word (bit 0: a Top-k segment emitted a wrong number of entries). */
int compams_check_status(compams_handle h, uint32_t* status_word);

/*
 * Per-kernel timing with CUDA events on the handle's stream.
 *   compams_set_profiling(h, mask): bit k of mask enables an event pair around every launch of
 *     kernel k (compams_kernel) in later steps; 0 disables. Timing state is reset.
 *   compams_get_kernel_time(h, k, &ms, &launches): synchronises the stream and returns the summed
 *     device time and launch count of kernel k since profiling was enabled.
 * At most 4096 launches are recorded between two resets; later ones are not timed.
 */
int compams_set_profiling(compams_handle h, uint32_t kernel_mask);
int compams_get_kernel_time(compams_handle h, int32_t kernel, double* total_ms, int64_t* launches);

/* Number of kernel launches the handle has enqueued since creation (all kernels, all steps). */
int64_t compams_launch_count(compams_handle h);

/*
 * compams_blocksign_sweep_static - the Block-Sign sweep for callers that cannot allocate device
 * memory (the paper has no counterpart: this is a packaging of the same arithmetic, not a step
 * of its algorithms).
 *
 * Who needs it: code that runs where cudaMalloc is not an option - inside another framework's
 * allocator or memory-pool callback, in a process whose device memory was partitioned up front,
 * or on a latency-critical path where the device-wide synchronisation of an allocation is not
 * acceptable. compams_create allocates; this call does not: it calls no cudaMalloc, cudaFree or
 * allocating library routine, and takes every input and output from the caller. Its only scratch
 * (per-tile partial sums, per-worker arrival counters; 516 KiB) is a fixed array inside the
 * library's device image, held by every GPU that loads the library until the process exits.
 *
 * What it computes, for every worker i over ONE block covering all d coordinates: the corrected
 * gradient x_i = g_i + e_i (Algorithm 2, the corrected-gradient step), written over x_state; the sign bit of every x_ij;
 * and the scale ||x_i||_1 / d (Definition 2). The residual update is deferred exactly as in
 * compams_step: with deferred != 0, x_state holds the PREVIOUS call's x and scales_prev that call's
 * scales, and e_i = x_prev - sign(x_prev) * scale_prev is formed on the fly; with deferred == 0,
 * x_state holds e itself (all zeros before the first step) and scales_prev is not read.
 *
 *   grads        device; [n, d] fp32 packed, 4-byte aligned; read only.
 *   x_state      device; [n, d] fp32 packed, 4-byte aligned; in: e or the previous x; out: x.
 *   scales_prev  device; [n] fp32; read when deferred != 0 (may be null otherwise). Must not alias scales_out.
 *   scales_out   device; [n] fp32; receives the scales.
 *   sign_bits    device; [n, ceil(d/32)] uint32; bit (j % 32) of word j / 32 of row i = sign bit of x_ij;
 *                unused high bits of a row's last word are 0.
 *   n, d         1 <= n <= 1024, 1 <= d < 2^31, and n * ceil(d / 8192) <= 65536
 *                (compams_blocksign_sweep_static_limits returns the two caps); beyond that the call
 *                does nothing and returns COMPAMS_ERR_TOO_LARGE.
 *   cuda_stream  a cudaStream_t passed as void* (null = default stream); the work is enqueued there
 *                and the call returns without synchronising.
 *
 * The first call on each device (with that device current) looks up the scratch array's device
 * address once; make that first call before starting any stream capture. Every call shares the one
 * array, which keeps the last call's contents (the counters are cleared at the start of each call):
 * calls whose device work overlaps in time - two streams, two threads - race on it, so serialise them.
 * Errors: INVALID_ARG (null / misaligned pointer, n or d out of range), TOO_LARGE, CUDA.
 */
int compams_blocksign_sweep_static(const float* grads, float* x_state, const float* scales_prev, float* scales_out,
                                   uint32_t* sign_bits, int32_t n, int64_t d, int32_t deferred, void* cuda_stream);
int compams_blocksign_sweep_static_limits(int64_t* max_workers, int64_t* max_tiles);

/* Static strings (never null). */
const char* compams_error_string(int status);
const char* compams_kernel_name(int32_t kernel);
/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char* compams_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* COMPAMS_H */
