/*
 * bmgd.h -- C ABI of the buffered mini-batch gradient descent (BMGD) library for NVIDIA B200.
 *
 * The library runs the computation step of BMGD (paper, Section 2.1 and Algorithm 1, inner
 * loops): T rounds of freshly shuffled mini-batch gradient descent, Eq. (2.1), over one
 * buffer that is resident in GPU memory, while the buffering step (Section 2.1, first bullet)
 * copies the next buffer from pinned host memory behind it.
 *
 * Vocabulary (paper, Section 2.2): the sample has N rows (X_i in R^p, Y_i); a pass over the
 * sample ("iteration") visits K buffers of N0 = ceil(N/K) rows; a round ("buffer epoch")
 * visits the M = ceil(rows/n) mini-batches of a fresh random partition of the buffer; one
 * step is  theta <- theta - alpha * (1/|S|) * sum_{i in S} grad l(X_i, Y_i; theta).
 * theta is carried from step to step, round to round and call to call.
 *
 * Conventions
 *   - Every function returns BMGD_OK (0) or a negative bmgd_status.  Nothing aborts, throws
 *     or traps.  Errors raised by a kernel (a bounded wait that ran out) surface at the next
 *     call that synchronises: bmgd_sync, bmgd_get_theta, bmgd_get_stats.
 *   - "host" pointers are CPU memory, "dev" pointers are memory of the handle's GPU.
 *   - A handle is not thread-safe.  Calls on one handle must come from one thread at a time.
 *   - Row layout: X is row-major [rows][p] in the storage type; y is [rows] (the parameter
 *     type for linear and logistic, int32 class labels for softmax).  theta is
 *     [Rc][p][C] row-major in the parameter type.
 */
#ifndef BMGD_H
#define BMGD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bmgd bmgd_t;

/* Per-sample loss.  Linear: gradient (x.theta - y) x, i.e. Eq. (3.1) without a factor 2.
 * Logistic: (sigmoid(x.theta) - y) x with y in {0,1} (Section 3.2.3, b' = sigmoid).
 * Softmax: outer(x, softmax(x W) - e_y), W in R^{p x C}; the C-class extension of the
 * logistic case (the paper itself stops at generalised linear models). */
enum { BMGD_LOSS_LINEAR = 0, BMGD_LOSS_LOGISTIC = 1, BMGD_LOSS_SOFTMAX = 2 };

/* Storage / arithmetic: fp64 rows and parameters; fp32 rows and parameters; bf16 rows with
 * fp32 parameters (softmax only). */
enum { BMGD_F64 = 0, BMGD_F32 = 1, BMGD_BF16X_F32W = 2 };

typedef enum {
    BMGD_OK = 0,
    BMGD_ERR_ARG = -1,           /* a null pointer, a size out of range, a bad enum */
    BMGD_ERR_ALLOC = -2,         /* device or host memory could not be had */
    BMGD_ERR_CUDA = -3,          /* a CUDA runtime call failed; see bmgd_last_cuda_error */
    BMGD_ERR_CAPACITY = -4,      /* more rows than a slot holds, or a workspace too small */
    BMGD_ERR_TIMEOUT = -5,       /* a device-side wait gave up; the results of that call are void */
    BMGD_ERR_NONFINITE = -6,     /* theta holds an Inf or a NaN (learning rate too large) */
    BMGD_ERR_LAUNCH = -7,        /* the grid cannot be made co-resident on this GPU */
    BMGD_ERR_UNIMPLEMENTED = -8, /* this combination of loss, type and shape has no kernel */
    BMGD_ERR_STATE = -9          /* slot not loaded, or call out of order */
} bmgd_status;

enum {
    BMGD_FLAG_FIXED_PARTITION = 1u, /* reuse round 0's partition in every round: the fixed-partition
                                       assumption under which Eq. (3.1)-(3.3) are derived */
    BMGD_FLAG_NO_SLOTS = 2u,        /* allocate no buffer slots: only bmgd_run_rounds_resident is used */
    BMGD_FLAG_TIMING = 4u,          /* record CUDA events round every launch and copy (bmgd_get_stats) */
    BMGD_FLAG_SOFTMAX_CUDA_CORES = 8u /* softmax: run the two contractions on the CUDA cores, not the tensor cores
                                       (same bf16 inputs; for cross-checking the tensor-core path) */
};

/* Everything bmgd_create cannot say.  Fill with bmgd_config_init, then change fields. */
typedef struct bmgd_config {
    int64_t N;                /* rows in the whole sample */
    int32_t p;                /* predictors per row */
    int32_t K;                /* buffers per pass; a slot holds N0 = ceil(N/K) rows */
    int32_t loss;             /* BMGD_LOSS_* */
    int32_t dtype;            /* BMGD_F64 / BMGD_F32 / BMGD_BF16X_F32W */
    int32_t C;                /* classes, softmax only (>= 2); otherwise 1 */
    int32_t Rc;               /* replicate chains: independent theta's, distinct shuffles, same buffer (any loss) */
    int32_t device;           /* CUDA device ordinal; -1 = the calling thread's current device */
    uint32_t flags;           /* BMGD_FLAG_* */
    void*   workspace;        /* dev memory, 256-byte aligned, owned by the caller and kept alive until
                                 bmgd_destroy; NULL = the library allocates and frees its own */
    int64_t workspace_bytes;  /* size of workspace; at least bmgd_workspace_bytes() */
    void*   compute_stream;   /* cudaStream_t the kernels run on; NULL = a stream the library creates */
    double  timeout_ms;       /* bound on any single device-side wait; <= 0 selects 2000 ms */
    /* Launch shape; 0 = chosen by the library.  A chain is worked on by ctas_per_chain CTAs
     * (a multiple of cluster_size); the rows of a mini-batch are split among them. */
    int32_t cluster_size;     /* CTAs per thread-block cluster: 1, 2, 4, 8 or 16 */
    int32_t ctas_per_chain;
    int32_t threads_per_cta;  /* linear/logistic: threads that compute, a multiple of 32 from 256 to 512 (softmax: fixed) */
    int32_t pipeline_depth;   /* row-prefetch stages held in shared memory: 2 to 8 (fewer where shared memory, or the
                                 warps a CTA has room for, do not allow as many: bmgd_get_stats reports what ran) */
    int32_t subpasses_per_stage; /* a stage holds this many sweeps of the CTA over its rows: 1, 2, 4, ... 32 */
    int32_t producer_warps;   /* linear/logistic: extra warps per CTA that only evaluate the shuffle and fetch rows: 1 to 8
                                 (rows that are not fetched by four-row gathers, i.e. not 16-byte multiples or wider than 256
                                 values, get a multiple of pipeline_depth of them: the value is rounded to one) */
    int32_t lanes_per_row;    /* linear/logistic: lanes that share one row in the inner loop: 4, 8, 16 or 32, if the row size has
                                 a kernel built that way */
    int32_t first_chain;      /* shuffle id of this handle's first chain: chain c of the handle draws the partitions of
                                 chain first_chain + c, so the chains of one job can be spread over several handles (one
                                 per GPU) and give, bit for bit, what one handle with all of them gives; default 0 */
    int32_t reserved[4];      /* must be zero */
} bmgd_config;

typedef struct bmgd_stats {
    int64_t launches;          /* kernels launched by bmgd_run_rounds* so far */
    int64_t steps;             /* mini-batch steps taken, summed over chains */
    int64_t sample_grads;      /* per-sample gradients evaluated, summed over chains */
    int64_t h2d_bytes;         /* bytes copied by bmgd_load_buffer */
    double  kernel_ms;         /* device time inside the step kernels (BMGD_FLAG_TIMING) */
    double  h2d_ms;            /* device time of the buffer copies (BMGD_FLAG_TIMING) */
    int32_t grid_ctas;         /* shape of the last launch */
    int32_t cluster_size;
    int32_t ctas_per_chain;
    int32_t threads_per_cta;   /* all warps of a CTA, those that only fetch rows included */
    int32_t pipeline_depth;
    int32_t smem_bytes;
    int32_t chains_in_flight;  /* chains worked on at the same time in the last launch */
    int32_t subpasses_per_stage;
} bmgd_stats;

/* Defaults: F32, linear, C = 1, Rc = 1, current device, two slots, library-owned memory. */
void bmgd_config_init(bmgd_config* cfg);

/* Device bytes a handle made from cfg needs (slots, theta, exchange buffers, status words). */
int bmgd_workspace_bytes(const bmgd_config* cfg, int64_t* bytes);

/*
 * Make a handle for a sample of N rows with p predictors, read in K buffers (Section 2.2),
 * for the given loss in fp32 with theta = 0 (Algorithm 1's initial value; use bmgd_set_theta
 * for another).  Allocates two slots of ceil(N/K) rows, theta and small exchange buffers on
 * the current device.  *out is set only on success and is released by bmgd_destroy.
 */
int bmgd_create(int64_t N, int32_t p, int32_t K, int32_t loss, bmgd_t** out);
int bmgd_create_ex(const bmgd_config* cfg, bmgd_t** out);
int bmgd_destroy(bmgd_t* h);

/*
 * Buffering step (Section 2.1, first bullet; Algorithm 1 line 3): start copying one buffer,
 * `rows` rows of host_x [rows][p] and host_y [rows], into the next free slot, asynchronously on
 * `stream` (a cudaStream_t owned by the caller; NULL = the legacy default stream).  The copy
 * first waits, on the stream, until the kernel that last read that slot has finished, so it
 * can be issued while an earlier buffer is still being computed on.  *slot receives the slot
 * id.  The host arrays must stay valid until the copy has run (bmgd_sync, or a
 * synchronisation of `stream`); they must be pinned for the copy to overlap with compute.
 * Errors: BMGD_ERR_CAPACITY if rows exceeds ceil(N/K); BMGD_ERR_STATE without slots.
 */
int bmgd_load_buffer(bmgd_t* h, const void* host_x, const void* host_y, int64_t rows,
                     void* stream, int32_t* slot);

/*
 * Computation step (Section 2.1, second bullet; Algorithm 1 lines 6-12; Eq. (2.1)): `rounds`
 * rounds over the buffer in `slot`, mini-batches of batch_size rows (the last one of a round
 * may be shorter and is averaged by its own size), learning rate lr, for every chain.  Round t
 * of chain c uses the partition keyed by (seed, c, t).  Asynchronous on the compute stream;
 * waits on-stream for the slot's copy.  theta is updated in place on the device.
 * Softmax handles (bf16 rows, fp32 W): at most 16 classes, p a multiple of 8 up to 3072 (any batch_size: a
 * mini-batch of more than 256 rows is taken in tiles of 256); other shapes return BMGD_ERR_UNIMPLEMENTED.
 */
int bmgd_run_rounds(bmgd_t* h, int32_t slot, int32_t rounds, int32_t batch_size, double lr,
                    uint64_t seed);

/* The same computation on a buffer the caller already holds in device memory (dev_x [rows][p],
 * dev_y [rows], 16-byte aligned); rows may exceed ceil(N/K).  The arrays must stay valid
 * until the compute stream has passed the call. */
int bmgd_run_rounds_resident(bmgd_t* h, const void* dev_x, const void* dev_y, int64_t rows,
                             int32_t rounds, int32_t batch_size, double lr, uint64_t seed);

/*
 * The paper has no counterpart to this call; it exists for callers that must not allocate.
 *
 * Some programs cannot call cudaMalloc where they need this library: a plugin running inside
 * another framework's memory budget, a service that fixed its device memory at start-up and
 * runs with the allocator locked, a step of a latency-critical loop where the implicit
 * device-wide synchronisation of an allocation is not acceptable.  bmgd_create_ex always
 * needs device memory (its own or a caller's workspace) and host memory for the handle.
 * This call needs neither: the scratch of the step kernel (the packets through which
 * thread-block clusters exchange partial gradients, and the status words) sits in a fixed
 * array of BMGD_NOALLOC_SCRATCH_BYTES that is part of the library image, so every GPU on
 * which the library is used holds that much from the first use until the process exits.
 * No cudaMalloc, cudaFree or other allocating routine is called.
 *
 * It runs `rounds` rounds over the buffer dev_x [rows][p], dev_y [rows] exactly as
 * bmgd_run_rounds_resident does (same kernels, same shuffle, same launch-shape rules at their
 * defaults) for the least-squares and logistic losses in BMGD_F32 or BMGD_F64, on the calling
 * thread's current device, ordered on `stream` (a cudaStream_t; NULL = the legacy default
 * stream).  dev_theta [Rc][p] is the caller's: it is read as the starting value and holds the
 * result.  The call returns after the kernel has finished: it synchronises `stream` itself (that is how
 * it reads the kernel's status words back), so it cannot run inside a stream capture.  Device-side
 * waits are bounded by a fixed 2000 ms (a handle's timeout_ms has no counterpart here); a wait that gives
 * up returns BMGD_ERR_TIMEOUT from this very call.
 *
 * Limits and sharing: p must not exceed BMGD_NOALLOC_MAX_P, else BMGD_ERR_CAPACITY is returned
 * and nothing runs.  All calls on one GPU, from any thread or stream, use the same array; it
 * keeps the contents of the previous call, so each call first clears the part it uses.  Two
 * calls that overlap in time on one GPU would race on it: issue them one after the other.
 * The first call on each device also looks up the array's device address (cudaGetSymbolAddress, once
 * per device, with that device current).
 */
#define BMGD_NOALLOC_MAX_P 256
#define BMGD_NOALLOC_SCRATCH_BYTES (256 + 2 * 160 * BMGD_NOALLOC_MAX_P * 2 * 8)
int bmgd_run_rounds_noalloc(const void* dev_x, const void* dev_y, int64_t rows, int32_t p, int32_t loss,
                            int32_t dtype, int32_t Rc, void* dev_theta, int32_t rounds, int32_t batch_size,
                            double lr, uint64_t seed, void* stream);

/* Wait for everything issued on the compute stream; report a device-side error if one was raised. */
int bmgd_sync(bmgd_t* h);

/* Synchronise, then copy theta [Rc][p][C] to out_host (bytes must equal its exact size in the
 * parameter type).  Returns BMGD_ERR_NONFINITE (after copying) if a value is Inf or NaN. */
int bmgd_get_theta(bmgd_t* h, void* out_host, int64_t bytes);
/* Synchronise, then overwrite theta from host memory of the same shape: a non-zero initial
 * value (Algorithm 1, "Require"), or resuming a run from a saved estimate. */
int bmgd_set_theta(bmgd_t* h, const void* host, int64_t bytes);

/*
 * Update rule of the computation step (Section 4.3: the buffering idea "combined with" other gradient-based rules,
 * BNAG and BAdam beside BMGD; Section 4.2 trains its logistic model with Adam).  With g the mean gradient of the
 * mini-batch and lr the step's learning rate:
 *   BMGD_OPT_SGD       theta <- theta - lr g                                   (Eq. (2.1); the default)
 *   BMGD_OPT_NESTEROV  v <- a v - lr g;  theta <- theta + a v - lr g           (a = momentum, 0 <= a < 1)
 *   BMGD_OPT_ADAM      m <- a m + (1-a) g;  v <- b v + (1-b) g^2;  t <- t + 1;
 *                      theta <- theta - lr (m / (1-a^t)) / (sqrt(v / (1-b^t)) + eps)   (Kingma & Ba 2014, Algorithm 1)
 * The state (v; or m, v and t) lives beside theta on the device, one copy per chain, is carried from call to call
 * like theta, and is set to zero by this call, which is ordered after the launches already issued.  Linear and
 * logistic losses; BMGD_ERR_UNIMPLEMENTED for softmax handles.  BMGD_ERR_ARG for values out of range.
 */
enum { BMGD_OPT_SGD = 0, BMGD_OPT_NESTEROV = 1, BMGD_OPT_ADAM = 2 };
int bmgd_set_optimizer(bmgd_t* h, int32_t kind, double a, double b, double eps);

/*
 * Learning rate of each update (Section 4.4: alpha_{r,j} = 0.025 + 0.025 cos(j pi / TMK) for the j-th update of
 * every pass r, initial value 0.05).  BMGD_LR_CONSTANT: the lr argument of bmgd_run_rounds, unchanged (the default).
 * BMGD_LR_COSINE: lr (1/2 + 1/2 cos(j pi / J)) for the j-th update, j = 1..J, of a pass of J = updates_per_pass
 * updates (T M K in the paper's notation); the count runs on from call to call and starts again after J updates
 * and when this function is called.  The paper's warm-up has no stated length and is left to the caller (lr is a
 * per-call argument).  Linear and logistic losses.
 */
enum { BMGD_LR_CONSTANT = 0, BMGD_LR_COSINE = 1 };
int bmgd_set_lr_schedule(bmgd_t* h, int32_t kind, int64_t updates_per_pass);

/* Change the bound on any single device-side wait of later launches (cfg.timeout_ms at creation): a wait that
 * lasts longer gives up, the launch ends early without writing theta back, and the next synchronising call returns
 * BMGD_ERR_TIMEOUT once; the handle stays usable.  <= 0 selects 2000 ms.  A bound below one microsecond makes every
 * wait that does not succeed at its first look give up (for testing the error path without hanging a GPU). */
int bmgd_set_timeout(bmgd_t* h, double timeout_ms);

/* Synchronise and fill *out. */
int bmgd_get_stats(bmgd_t* h, bmgd_stats* out);

/* Write the shuffle of one round, out_host[j] = pi(j) for j in [0, N0), computed by the same
 * device function the step kernels use.  For checking the partition bit for bit. */
int bmgd_debug_perm(bmgd_t* h, uint64_t seed, uint32_t chain, uint32_t round, uint32_t N0,
                    uint32_t* out_host);

/*
 * Partition of the whole sample into buffers (Algorithm 1, line 2: a fresh random partition {S_r,1..S_r,K} at the
 * top of every pass r).  The partition of pass `pass` under `seed` is the same keyed bijection pi as the per-round
 * shuffle, taken over [0, N) with the chain word 0xFFFFFFFF and the pass number as the round word; buffer k holds,
 * in this order, rows pi(j) for k*N0 <= j < min((k+1)*N0, N), N0 = ceil(N/K).
 *
 * bmgd_partition_index writes pi(j) to *row.  bmgd_gather_buffer is the CPU side of the buffering step (Algorithm 1,
 * line 3, "CPU starts preparing buffered data"): with `threads` host threads (<= 0: all hardware threads) it copies
 * the rows of buffer k from host_x [N][row_bytes] and host_y [N][y_bytes] into stage_x, stage_y (at least N0 rows;
 * pinned memory if they are handed to bmgd_load_buffer next) and writes the row count to *rows_out.  Pure host
 * code: no GPU, no handle; safe to run from another thread while kernels and copies of earlier buffers are in flight.
 * Errors: BMGD_ERR_ARG for null pointers or sizes out of range (N up to 2^31 - 1).
 */
int bmgd_partition_index(uint64_t seed, uint32_t pass, int64_t N, int64_t j, int64_t* row);
int bmgd_gather_buffer(const void* host_x, const void* host_y, int64_t N, int64_t row_bytes, int64_t y_bytes,
                       int32_t K, uint64_t seed, uint32_t pass, int32_t k, void* stage_x, void* stage_y,
                       int32_t threads, int64_t* rows_out);

/* Latency probe of the computation step: launch, on the compute stream, the step
 * kernel's own synchronisation structure for a buffer of `rows` rows, `rounds` rounds and mini-batches of
 * batch_size rows, in the launch shape bmgd_run_rounds would choose, with every ring hand-over, barrier, packet
 * exchange between CTAs and update of a step, but without fetching or multiplying a single row (the gradient is
 * zero, so theta, the update rule's state and the step counters stay as they are).  Timed like any launch under
 * BMGD_FLAG_TIMING (bmgd_get_stats: launches, kernel_ms).  Its time per step is the floor that the dependency of
 * each step on the one before (Eq. (2.1)) puts under the step time of a single chain, whatever the memory system
 * delivers. */
int bmgd_debug_null_rounds(bmgd_t* h, int64_t rows, int32_t rounds, int32_t batch_size);

/* Launch, on the compute stream, a one-thread kernel that waits with the step kernels' bounded-wait protocol for
 * something that never happens, with a budget of budget_ms (at most 1000).  The wait gives up, the kernel returns,
 * and the next synchronising call reports BMGD_ERR_TIMEOUT once; the handle stays usable.  For testing the error
 * path without hanging or faulting a GPU.  Not for softmax handles. */
int bmgd_debug_wait_timeout(bmgd_t* h, double budget_ms);

/* Text for a bmgd_status; never NULL. */
const char* bmgd_strerror(int status);
/* cudaError_t of the last failed runtime call on this handle (0 if none). */
int bmgd_last_cuda_error(const bmgd_t* h);
/* ABI version: major * 1000 + minor. */
int bmgd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BMGD_H */
