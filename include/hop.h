/*
 * hop.h -- C ABI of the Hop hot path (heterogeneity-aware decentralized SGD, arXiv 1902.01064)
 * for N simulated workers whose parameter replicas all live in one GPU's memory.
 *
 * One logical iteration ("level" k) for all workers is: every worker i that executes iteration k
 * computes a minibatch gradient on x_{k,i} (Fig. alg0 step 1; the "parallel approach" of
 * Section 3.2: the gradient is taken before the Reduce), averages the in-neighbour versions the
 * queue protocol let it consume (Recv/Reduce of Fig. alg4 and Fig. alg3, weights of Eq. 1 or
 * Eq. 2) and applies the gradient (Fig. alg0 step 3).  Which (in-neighbour, version) pairs are
 * consumed is an integer "trace" produced on the host by a deterministic simulation of the
 * protocol (update queues Section 4.1, token queues Section 4.2, backup workers Section 4.3,
 * bounded staleness Section 4.4, skipping iterations Section 5).
 *
 * Conventions
 *   - Every function returns 0 (HOP_OK) or a negative hop_status; hop_last_error() gives a
 *     human-readable message for the last failure on that context (or of hop_create /
 *     hop_trace_create when passed NULL).  Nothing throws, aborts or traps.
 *   - "host" pointers are ordinary CPU memory, read or written before the call returns.
 *     "device" pointers are CUDA device memory owned by the caller; the context only borrows
 *     them and they must stay valid until hop_destroy or the next bind call.
 *   - Work is enqueued on the CUDA stream given to hop_bind_buffers and is asynchronous unless
 *     stated otherwise.  A context is not thread-safe.
 *   - The library keeps small device tables of its own (the uploaded trace, per-minibatch hinge
 *     coefficients); they are allocated in hop_load_trace / hop_bind_svm_* / hop_step_host and
 *     freed in hop_destroy.  hop_step itself allocates nothing.
 *   - There is no CPU fallback: device entry points fail with HOP_E_CUDA when no GPU is usable.
 *
 * Data layout in device memory (all float32, row-major, the parameter index fastest):
 *   X[N][s+1][P]  ring of s+1 versions per worker; version v of worker i sits in slot v mod (s+1)
 *                 (Section 6: one queue per iteration slot, index mod(iter, #queues)).
 *   M[N][P]       momentum buffers (only with momentum != 0)
 *   G[N][P]       dense gradients of the current level (not used by the CSR SVM mode)
 */
#ifndef HOP_B200_H
#define HOP_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hop_ctx hop_ctx;
typedef struct hop_trace hop_trace;

typedef enum hop_status {
    HOP_OK = 0,
    HOP_E_ARG = -1,         /* null pointer, negative size, unknown option ...                    */
    HOP_E_GRAPH = -2,       /* missing self-loop, duplicate edge, b >= |N_in(i)|, max_skip > s+1  */
    HOP_E_TRACE = -3,       /* trace record violates the protocol (see hop_load_trace)            */
    HOP_E_STATE = -4,       /* call out of order: no buffers bound, no trace loaded, past the end */
    HOP_E_DEADLOCK = -5,    /* the simulated protocol cannot make progress                        */
    HOP_E_CUDA = -6,        /* a CUDA runtime call failed (message has the CUDA error string)     */
    HOP_E_DEVICE = -7,      /* a kernel reported a failed internal check (see hop_read_status)    */
    HOP_E_UNSUPPORTED = -8  /* combination not implemented (e.g. momentum with the CSR SVM mode)  */
} hop_status;

/* Per (level, worker) operation in a trace. */
typedef enum hop_op {
    HOP_OP_IDLE = 0,    /* the worker skipped this iteration (Section 5)                          */
    HOP_OP_NORMAL = 1,  /* Compute + Recv + Reduce + Apply of Fig. alg2                           */
    HOP_OP_JUMP = 2     /* Recv(k) + Reduce of the worker's current parameters before a jump to   */
                        /* iteration k+1 (Section 5); no gradient                                  */
} hop_op;

/* Reduce weights. UNIFORM: 1/|consumed| (Fig. alg4 Reduce; Eq. 1 when everything is consumed).
 * STALE_LINEAR: numerator Iter(u) - (k - s) + 1, normalised (Eq. 2). */
typedef enum hop_weight_mode { HOP_W_UNIFORM = 0, HOP_W_STALE_LINEAR = 1 } hop_weight_mode;

/* Which usable updates enter the Reduce under bounded staleness (s > 0).  An in-neighbour is usable at
 * iteration k when the newest update ever dequeued from it has iteration >= k - s; that decides blocking
 * in both modes (Section 4.4: an older update still inside the bound needs no new arrival).
 * NEW_ONLY (default, the printed rule): only updates this Recv itself dequeued are reduced -- Eq. 2 sums over
 * the in-neighbours whose update received in iteration k is usable, and Fig. alg3's Recv appends an update
 * only when the newest iteration among what the call dequeued is inside the bound.  A neighbour that has not
 * advanced since the worker's previous Recv adds no term; the own update is always new.
 * REUSE: such a neighbour's last update is reduced again with the smaller weight Eq. 2 gives its age, so every
 * usable in-neighbour contributes at every iteration.  With s = 0 both coincide. */
typedef enum hop_stale_reduce { HOP_STALE_NEW_ONLY = 0, HOP_STALE_REUSE = 1 } hop_stale_reduce;

/* What Recv keeps once |N_in(i)| - N_buw(i) in-neighbours are usable.  AT_LEAST: every usable update
 * (Fig. alg4: the needed ones, then whatever else is queued for that iteration).  EXACT: exactly
 * |N_in(i)| - N_buw(i): the own update plus the neighbours whose first usable update was sent
 * earliest (what a FIFO dequeue of that many entries returns), ties by worker id. */
typedef enum hop_backup_mode { HOP_BACKUP_AT_LEAST = 0, HOP_BACKUP_EXACT = 1 } hop_backup_mode;

/* Loss of the linear model in the SVM modes: coef_r = d loss / d margin_r.
 * HINGE: -y_r/B if y_r * margin_r < 1 else 0.   LOG: -y_r / (B * (1 + exp(y_r * margin_r))). */
typedef enum hop_loss { HOP_LOSS_HINGE = 0, HOP_LOSS_LOG = 1 } hop_loss;

/* Order of the five operations inside an iteration (Section 3.2).  PARALLEL: Send x_k, Compute on x_k, Recv,
 * Reduce, Apply: x_{k+1} = Reduce(versions) - eta * d.  SERIAL: Compute, Apply, Send, Recv, Reduce:
 * x'_k = x_k - eta * d replaces version k in the ring before anyone consumes it, x_{k+1} = Reduce(versions).
 * hop_sim_run follows the same order: in the serial approach the update of iteration k becomes visible to the
 * out-neighbours when Compute(k) ends, in the parallel approach when iteration k is entered. */
typedef enum hop_approach { HOP_APPROACH_PARALLEL = 0, HOP_APPROACH_SERIAL = 1 } hop_approach;

/* Where the gradient of a level comes from. */
typedef enum hop_grad_mode {
    HOP_GRAD_EXTERNAL = 0,   /* the caller fills G before each hop_step                            */
    HOP_GRAD_SYNTHETIC = 1,  /* G[i][p] = sigma * normal(seed, i, k, p): Philox4x32-10 with counter */
                             /* (p/4, i, k, 6), key = seed, Box-Muller on 23-bit uniforms          */
    HOP_GRAD_SVM_DENSE = 2,  /* hinge-loss linear SVM, dense rows (hop_bind_svm_dense)             */
    HOP_GRAD_SVM_CSR = 3     /* hinge-loss linear SVM, CSR rows (hop_bind_svm_csr)                 */
} hop_grad_mode;

/* AUTO: TENSOR for dense levels (>= 32 active workers consuming >= 32 updates each, N <= 128, P % 128 == 0; with
 * momentum or weight decay a pre-pass first turns G into the update direction in place, so a G the caller supplied
 * is overwritten), else BULK (STAGED only when P % 4 != 0 and the level's tables exceed 32 KB of shared
 * memory).  hop_level_stats reports the kernel each level was planned with. */
typedef enum hop_mix_kernel {
    HOP_MIX_AUTO = 0,
    HOP_MIX_STAGED = 1,      /* column tile staged in shared memory by cp.async, two stages; any P */
    HOP_MIX_BULK = 2,        /* same, slices fetched by bulk copies, producer and consumer warps;  */
                             /* any P (with P % 4 != 0 the rows are not 16-byte aligned: each is   */
                             /* fetched from the boundary below it and read back with scalar loads) */
    HOP_MIX_TENSOR = 3       /* dense graphs: W_k * X on tcgen05 tensor cores, 3xTF32              */
} hop_mix_kernel;

typedef enum hop_option {
    HOP_OPT_MAX_IG = 1,       /* token-queue bound max_ig >= 1 (Section 4.2); 0 = no token queues;  */
                              /* default max(1, s)                                                  */
    HOP_OPT_LR = 2,           /* learning rate eta (default 0.1)                                    */
    HOP_OPT_MOMENTUM = 3,     /* mu; m <- mu*m + g, x <- mix - eta*m; buffers local (default 0)     */
    HOP_OPT_WEIGHT_MODE = 4,  /* hop_weight_mode (default UNIFORM)                                  */
    HOP_OPT_GRAD_MODE = 5,    /* hop_grad_mode (default EXTERNAL)                                   */
    HOP_OPT_GRAD_SEED = 6,    /* integer < 2^53                                                     */
    HOP_OPT_GRAD_SIGMA = 7,   /* default 1e-3                                                       */
    HOP_OPT_MIX_KERNEL = 8,   /* hop_mix_kernel (default AUTO)                                      */
    HOP_OPT_COL_OFFSET = 9,   /* global index of local parameter 0 when P is a shard of a larger    */
                              /* vector (multiple of 4); only the synthetic gradient reads it       */
    HOP_OPT_USE_GRAPH = 10,   /* hop_run may replay a captured CUDA graph (default 1)               */
    HOP_OPT_BACKUP_MODE = 11, /* hop_backup_mode (default AT_LEAST)                                 */
    HOP_OPT_NOTIFY_ACK = 12,  /* 1: simulate the NOTIFY-ACK scheme of Section 3.3 (the paper's baseline)  */
                              /* instead of token queues: iteration k+1 is entered only once every   */
                              /* out-neighbour has reduced iteration k-1; max_ig is ignored          */
    HOP_OPT_WEIGHT_DECAY = 13,/* lambda >= 0: lambda * x_{k,i} is added to the gradient (Section 7.2 uses 1e-4 / 1e-7)  */
    HOP_OPT_LOSS = 14,        /* hop_loss of the SVM modes (default HINGE; the paper's runs used LOG, Section 7.2)    */
    HOP_OPT_APPROACH = 15,    /* hop_approach (default PARALLEL, the paper's choice, Section 3.2)                     */
    HOP_OPT_STALE_REDUCE = 16,/* hop_stale_reduce (default NEW_ONLY: Eq. 2 / Fig. alg3 as printed)                    */
    HOP_OPT_NVTX = 17,        /* 1: an NVTX range "hop level k" on the host timeline around each level's launches     */
    HOP_OPT_BACKUP_OF_WORKER = 1000 /* key = 1000 + i sets N_buw(i) of one worker (Fig. alg4)       */
} hop_option;

/* ---- context -------------------------------------------------------------------------------
 * Problem statement of Figs. alg1-alg4: graph G (in-neighbour lists in CSR form, self-loop
 * required at every node, Section 3.1), N workers, P parameters, staleness bound s >= 0
 * (max_staleness of Fig. alg3), backup workers b (N_buw, the same for every worker; must be
 * < |N_in(i)|), max_skip >= 0 = largest number of iterations skipped in one jump (0 disables
 * skipping; <= s+1 so that the jumper's parameters are still inside its version ring).
 * in_ptr[N+1] and in_idx[in_ptr[N]] are host arrays, copied.  Touches no GPU. */
int hop_create(hop_ctx** out, const int32_t* in_ptr, const int32_t* in_idx,
               int32_t N, int64_t P, int32_t s, int32_t b, int32_t max_skip);
int hop_destroy(hop_ctx* ctx);
const char* hop_last_error(const hop_ctx* ctx);
/* Options may be set at any time except between hop_step_begin and hop_step_end.  Every call drops the CUDA
 * graphs hop_run has cached.  With a trace loaded, a change of HOP_OPT_MOMENTUM (zero <-> non-zero),
 * HOP_OPT_WEIGHT_DECAY (zero <-> non-zero), HOP_OPT_APPROACH, HOP_OPT_GRAD_MODE or HOP_OPT_MIX_KERNEL plans and
 * uploads the loaded levels again (tile widths, kernel choice and the staged rows depend on them; this frees and
 * allocates the device tables and synchronises) and keeps the current level; if the trace cannot be planned
 * under the new value the call fails and the option keeps its old value.  The protocol options (max_ig, weight
 * mode, backup mode, stale-reduce mode, N_buw) act on hop_sim_run and on the validation of traces loaded later. */
int hop_set_option(hop_ctx* ctx, int key, double value);

/* ---- protocol simulation (host only, no GPU) --------------------------------------------------
 * ticks[N][iters] (host): Compute of worker i in iteration k lasts ticks[i*iters+k] >= 1 time
 * units; every other operation is instantaneous.  Runs Train() of Fig. alg2 for all workers with
 * Recv of Figs. alg3/alg4 and the skipping rule of Section 5 and returns the consumption trace.
 * HOP_E_DEADLOCK if no worker can move before all are finished. */
int hop_sim_run(hop_ctx* ctx, const uint64_t* ticks, int32_t iters, hop_trace** out);

/* A trace from caller-supplied host arrays (copied): op[levels*N]; ptr[levels*N+1] offsets into
 * nbr/ver/num (record of (k,i) = [ptr[k*N+i], ptr[k*N+i+1])); den[levels*N]. */
int hop_trace_create(hop_trace** out, int32_t levels, int32_t N, const int32_t* op,
                     const int64_t* ptr, const int32_t* nbr, const int32_t* ver,
                     const int32_t* num, const int32_t* den);
int hop_trace_dims(const hop_trace* t, int32_t* levels, int32_t* N, int64_t* entries,
                   uint64_t* makespan_ticks);
/* Copies the trace into caller arrays of the sizes given by hop_trace_dims (any may be NULL). */
int hop_trace_export(const hop_trace* t, int32_t* op, int64_t* ptr, int32_t* nbr, int32_t* ver,
                     int32_t* num, int32_t* den);
int hop_trace_destroy(hop_trace* t);

/* ---- device buffers ---------------------------------------------------------------------------
 * X, M, G: device pointers laid out as above, 16-byte aligned; M may be NULL when momentum is 0,
 * G may be NULL in CSR SVM mode.  cuda_stream is a cudaStream_t (NULL = default stream). */
int hop_bind_buffers(hop_ctx* ctx, float* X, float* M, float* G, void* cuda_stream);

/* Hinge-loss linear SVM without bias or regulariser: margin_r = a_r . x_{k,i};
 * coef_r = -y_r / batch if y_r * margin_r < 1 else 0; g = sum_r coef_r a_r.  The minibatch of
 * iteration k is rows [(k mod (rows_per_worker/batch)) * batch, +batch) of the worker's shard.
 * Dense: A[N][rows_per_worker][P], y[N][rows_per_worker] (device).  CSR: row_ptr[N*rows+1]
 * (global offsets), col, val, y (device).  Allocates N*batch floats of device scratch (a second bind frees
 * and reallocates it, synchronising the device, and drops the CUDA graphs hop_run has cached, since they hold
 * the old pointers). */
int hop_bind_svm_dense(hop_ctx* ctx, const float* A, const float* y,
                       int32_t rows_per_worker, int32_t batch);
int hop_bind_svm_csr(hop_ctx* ctx, const int64_t* row_ptr, const int32_t* col, const float* val,
                     const float* y, int32_t rows_per_worker, int32_t batch);

/* Validates every record on the host -- consumed neighbour in N_in(i), version in [k-s, k] and
 * actually produced, own update present, at least |N_in(i)| - b entries (with s > 0 under
 * HOP_STALE_NEW_ONLY: at least the own update), versions consumed over an edge never going back
 * (and never repeating under HOP_STALE_NEW_ONLY), positive numerators summing to den,
 * JUMP/IDLE consistent with the versions a worker holds -- then uploads the
 * per-level tables (cudaMalloc + H2D on the bound stream) and rewinds to level 0. */
int hop_load_trace(hop_ctx* ctx, const hop_trace* t);

/* Version `version` of worker `worker` (-1 = every worker) <- host_src[P]; synchronous. */
int hop_write_params(hop_ctx* ctx, int32_t worker, int32_t version, const float* host_src);
/* host_dst[P] <- version `version` (-1 = newest the worker holds after the executed levels) of
 * worker `worker`; synchronises the stream. */
int hop_read_params(hop_ctx* ctx, int32_t worker, int32_t version, float* host_dst);
/* Newest version worker holds after the levels executed so far. */
int hop_newest_version(hop_ctx* ctx, int32_t worker, int32_t* version);

/* Next level to execute (momentum buffers are not touched). */
int hop_set_level(hop_ctx* ctx, int32_t level);
/* Executes the next level k of the loaded trace for all N workers: gradient kernels on slot k,
 * then the fused gather-mix-update writing slot k+1, then (CSR SVM) the sparse apply.
 * Asynchronous; HOP_E_STATE past the end of the trace.
 * Ordering on the stream: the first kernel of a call waits for everything enqueued before the call; the kernels
 * of the call are ordered among themselves, except that the mix-update kernel may read X and M (which the
 * library's gradient kernels do not write) while the level's gradient kernel is still finishing -- it waits for
 * that kernel before it reads G and before it writes anything.  With HOP_GRAD_EXTERNAL every kernel is fully
 * ordered behind the caller's work. */
int hop_step(hop_ctx* ctx);
/* Split-phase form of hop_step for a parameter vector sharded by columns over several contexts (one per GPU):
 * mixing and the dense / synthetic gradients are separable by column, but an SVM margin a_r . x needs all columns.
 * hop_step_begin enqueues the gradient phase; in the SVM modes it stops after the partial margins over this
 * context's columns and returns their device address (double[N * batch], owned by the context; entry
 * [i * batch + r] for row r of worker i's minibatch) for the caller to sum across the shards -- e.g. one NCCL
 * all-reduce on the bound stream.  hop_step_end computes the coefficients from the summed margins and finishes the
 * level.  With one shard, begin + end equals hop_step.  In the other gradient modes *margins is NULL, *count 0. */
int hop_step_begin(hop_ctx* ctx, double** margins, int64_t* count);
int hop_step_end(hop_ctx* ctx);
/* Executes the next n_levels levels of the loaded trace.  When the bound stream is not the default
 * stream, the levels are captured once into a CUDA graph (cached per (first level, n_levels); dropped
 * by any bind / option / trace change) and replayed, which removes most of the per-kernel launch cost
 * that dominates small problems.  Falls back to a plain loop of hop_step on the default stream, while
 * timing is enabled, with HOP_GRAD_EXTERNAL, or with HOP_OPT_USE_GRAPH = 0.  Asynchronous.
 * Inside one call the CSR margin kernel of every level but the first may fetch its row data (row_ptr, col, val:
 * read-only to the library) while the previous level's last kernel is finishing. */
int hop_run(hop_ctx* ctx, int32_t n_levels);
/* Same for one level handed in from the host (streaming use: the protocol decides level by
 * level): validates the records, uploads them from a pinned staging buffer, executes the level,
 * copies the first probe_len floats of worker 0's new version into probe_dst (host, may be NULL)
 * and synchronises.  op[N], ptr[N+1], den[N]; nbr/ver/num as in hop_trace_create. */
int hop_step_host(hop_ctx* ctx, const int32_t* op, const int64_t* ptr, const int32_t* nbr,
                  const int32_t* ver, const int32_t* num, const int32_t* den,
                  float* probe_dst, int64_t probe_len);

/* Synchronises and returns the device-side error word.  Every wait inside the kernels (on a copy, on a free
 * stage, on the tensor pipeline) is bounded; a kernel that gives up records the first such event and returns, so
 * the context and the GPU stay usable.  0 = nothing happened (HOP_OK); otherwise HOP_E_DEVICE, the word has a code
 * in its top byte (1: mix_bulk_kernel, a tile's copies did not arrive; 2: mix_bulk_kernel, no stage became free;
 * 3: mix_dense_tc_kernel, a pipeline wait ran out; 4: only in the bounds-checked build of the library, an access
 * outside the bound buffers was refused) and a detail in the low 24 bits (tile index or site), and
 * hop_last_error names it.  The parameters written by that level are then undefined.  The word is sticky until
 * hop_clear_status. */
int hop_read_status(hop_ctx* ctx, int32_t* device_error_word);
/* 1 if this library is the bounds-checked build (compiled with -DHOP_CHECKED: global-memory sources of the mix kernels'
 * copies and the gathers / atomics of the CSR SVM kernels are tested against the bound buffers X, M, G; an access outside
 * them is refused and recorded as status code 4; hop_run does not replay graphs), else 0.  Touches no GPU. */
int hop_build_is_checked(void);
/* Resets the device-side error word (asynchronous on the bound stream). */
int hop_clear_status(hop_ctx* ctx);
/* Self-test of that mechanism: launches one warp that waits on a barrier nothing completes, gives up after `polls`
 * polls (1..65536, ~32 ns apart) and records code 1 with `detail`.  hop_read_status then reports HOP_E_DEVICE. */
int hop_selftest_bounded_wait(hop_ctx* ctx, int32_t polls, int32_t detail);

/* out[10] (host) for a level of the loaded trace: distinct consumed slices U_k, NORMAL records,
 * JUMP records, consumed entries sum_i |C_{i,k}|, tile width chosen, kernel chosen (hop_mix_kernel),
 * staged rows, algorithmic bytes of the mix-update kernel, tensor-core flops issued by the dense
 * path (0 for the other kernels), K padded to the MMA chunk (dense path). */
int hop_level_stats(hop_ctx* ctx, int32_t level, int64_t* out);
/* Per-kernel-class timing (tracing aid).  While enabled, hop_step / hop_step_host bracket each
 * kernel class with CUDA events on the bound stream.  hop_timing_read synchronises the stream and
 * returns, since the last read: ms[3] = {gradient kernels, mix-update kernel, sparse apply}, the
 * number of timed spans of each class, and the algorithmic bytes of the timed mix-update launches
 * (per level: every distinct consumed slice once + dense gradient once + result once, + momentum
 * read and write); then it resets the counters. */
int hop_timing_enable(hop_ctx* ctx, int32_t on);
int hop_timing_read(hop_ctx* ctx, double* ms, int64_t* spans, int64_t* mix_bytes);
/* Number of kernels launched by this context so far. */
int hop_launch_count(hop_ctx* ctx, int64_t* launches);

/* ---- allocation-free entry point (the paper has no counterpart) -------------------------------
 * For callers that are not allowed to allocate device memory while they run: code inside a
 * region where cudaMalloc is forbidden or would synchronise the device (a latency-critical loop,
 * a plugin hosted by a framework that owns the allocator, a process whose memory budget is fixed
 * at start-up).  It performs the hinge-loss SVM minibatch step of hop_bind_svm_csr + hop_step for
 * ONE parameter vector without any context: coef_r = -y_r/rows if y_r * (a_r . x) < 1 else 0,
 * then x_out[col] -= lr * coef_r * val for every stored element of the `rows` CSR rows.  x_out may
 * alias x when no mixing happens in between, or hold the mixed parameters.
 *
 * The per-row coefficients, which hop_step keeps in a cudaMalloc'ed buffer, are written to a
 * fixed array of HOP_STATIC_MAX_ROWS floats (64 KiB) inside the library image; every GPU that
 * loads the library carries it until the process exits.  The call makes no cudaMalloc / cudaFree
 * and calls no allocating library routine.  rows > HOP_STATIC_MAX_ROWS is rejected with
 * HOP_E_ARG and a message in errbuf.
 *
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.  All calls on a device share the
 * array and it keeps the previous call's coefficients (each call overwrites the rows it uses
 * before reading them, so nothing needs clearing); two calls whose kernels overlap on the GPU
 * (different streams) race on it -- serialise them.
 *
 * x, x_out: device float[P]; row_ptr: device int64[rows+1] offsets into col/val; col: device
 * int32 (each < P, not checked); val: device float; y: device float[rows] (+1/-1).  Asynchronous
 * on cuda_stream.  errbuf (host, may be NULL) receives a NUL-terminated message on failure. */
#define HOP_STATIC_MAX_ROWS 16384
int hop_svm_csr_sgd_static(const float* x, float* x_out, int64_t P, const int64_t* row_ptr,
                           const int32_t* col, const float* val, const float* y, int32_t rows,
                           float lr, void* cuda_stream, char* errbuf, int64_t errbuf_len);

#ifdef __cplusplus
}
#endif
#endif /* HOP_B200_H */
