/*
 * gnnpre — multi-hop feature aggregation  X_k = A^ X_{k-1}, k = 1..K, on one Blackwell GPU.
 *
 * C ABI of libgnnpre.so.  The library implements the block-wise precomputation of
 * arXiv 2207.12000, Section 3.2 ("Efficient Precomputation"):
 *   - the edge list E of the operator's support is cut into b disjoint, balanced sets
 *     ("Precomputation on GPU", Eq. 10; Algorithm 1, the split of S),
 *   - the feature matrix is cut into c column slabs (Algorithm 1, the split of X_prev),
 *   - (b, c) minimise b*c under a device-memory budget (Eq. 12),
 *   - every hop multiplies the previous hop (Algorithm 1's outer loop); all K hops are kept.
 * A^ is a constant linear filter fixed before precomputation (Section 3.1, "Limitation"):
 *   GCN_SYM    S = D~^{-1/2} (A + I) D~^{-1/2}           (Eq. 1)
 *   SAGE_MEAN  D^{-1} A, zero rows where D_i = 0
 *   GIN_SUM    A + (1 + eps) I, eps fixed by the caller
 *
 * Conventions
 *   - Every function returns a gnnpre_status_t (0 = success, negative = error); nothing
 *     throws or aborts across this boundary.  On error no output argument is valid unless
 *     stated otherwise.
 *   - "device" pointers are CUDA device addresses on the current device; "host" pointers are
 *     ordinary process addresses.  The library never takes ownership of a caller's buffer.
 *   - There is no CPU fallback: host-resident operands are streamed through the GPU.
 *   - Only sm_100 devices are accepted (GNNPRE_ERR_UNSUPPORTED_ARCH otherwise).
 *   - Logging: GNNPRE_LOG=1 in the environment prints one line per gnnpre_propagate call to stderr; GNNPRE_LOG=2
 *     also prints the timeline of every streamed call (each copy, and the first and last edge block of each
 *     compute job, in milliseconds since the call began).  Nothing is printed otherwise.
 */
#ifndef GNNPRE_H
#define GNNPRE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GNNPRE_OK = 0,
    GNNPRE_ERR_INVALID_ARG = -1,      /* NULL pointer, bad enum, bad size, b > |E| ... */
    GNNPRE_ERR_INVALID_CSR = -2,      /* see gnnpre_csr_t */
    GNNPRE_ERR_ALIGN = -3,            /* pointer not 16-byte aligned, or a leading dimension not a multiple of 4 */
    GNNPRE_ERR_OOM_DEVICE = -4,
    GNNPRE_ERR_OOM_HOST = -5,
    GNNPRE_ERR_BUDGET_TOO_SMALL = -6, /* Eq. 12 has no feasible (b, c) */
    GNNPRE_ERR_CUDA = -7,             /* a CUDA call failed; gnnpre_last_cuda_error() names it */
    GNNPRE_ERR_TIMEOUT = -8,
    GNNPRE_ERR_BUSY = -9,             /* the plan is already inside a propagate call */
    GNNPRE_ERR_UNSUPPORTED_ARCH = -10,
    GNNPRE_ERR_TOO_LARGE = -11        /* gnnpre_hop_static: the problem does not fit the fixed scratch array */
} gnnpre_status_t;

typedef enum { GNNPRE_OP_GCN_SYM = 0, GNNPRE_OP_SAGE_MEAN = 1, GNNPRE_OP_GIN_SUM = 2 } gnnpre_op_t;
typedef enum { GNNPRE_MEM_DEVICE = 0, GNNPRE_MEM_HOST = 1 } gnnpre_mem_t;

/*
 * The adjacency matrix A in {0,1}^{n x n} (Section 2) in CSR form, WITHOUT diagonal entries.
 *   rowptr[n+1] int64, rowptr[0] = 0, non-decreasing, rowptr[n] = nnz
 *   colidx[nnz] int32, 0 <= col < n < 2^31, strictly ascending inside a row, col != row
 * Both arrays live where `mem` says (both on the device, or both on the host; host arrays are
 * read fastest when page-locked).  Symmetry is the caller's business: degrees are row counts.
 * The arrays are only read during gnnpre_build_plan and may be released afterwards.
 */
typedef struct {
    int64_t n;
    int64_t nnz;
    const int64_t* rowptr;
    const int32_t* colidx;
    int32_t mem; /* gnnpre_mem_t */
} gnnpre_csr_t;

/* gnnpre_plan_opts_t.flags */
#define GNNPRE_FLAG_LAUNCH_PER_BLOCK 1u /* device-resident runs: one kernel launch per edge block instead of one per hop */
#define GNNPRE_FLAG_SKIP_VALIDATION 2u  /* trust the CSR contract (saves one pass over the graph) */
#define GNNPRE_FLAG_NO_BULK_COPY 4u     /* gather into registers for every width (default: rows of 68..128 columns
                                           are staged through shared memory by the bulk-copy engine); same bits */

typedef struct {
    int32_t op;              /* gnnpre_op_t */
    float gin_eps;           /* GIN_SUM only */
    int64_t feat_dim;        /* F: columns of X.  Work is done on whole groups of 4 columns: with F % 4 != 0 the
                                1..3 pad columns up to the next multiple of 4 (which ldx, ldo >= that multiple
                                make room for) are read from X and written to out[] with unspecified values */
    int64_t budget_bytes;    /* B_GPU of Eq. 12; 0 = the device's free memory at plan time */
    int32_t force_blocks;    /* b; 0 = solve Eq. 12 */
    int32_t force_col_slabs; /* c; 0 = solve Eq. 12 */
    int32_t segment_edges;   /* edges per warp-level segment; 0 = chosen from F */
    int32_t operands_mem;    /* gnnpre_mem_t: where X and out[] will live at propagate time; HOST makes
                                Eq. 12 count the library's four slab buffers (beta_X = 4) instead of two, and
                                raises an unforced c = 1 to c = 2 (F >= 128) and an unforced b = 1 to b = 8
                                (|E| >= 2^20) so that copies and kernels overlap */
    uint32_t flags;
    float teleport_alpha;    /* 0 = plain propagation X_k = A^ X_{k-1}; in (0, 1]: the personalised-PageRank power
                                iteration X_k = (1 - alpha) A^ X_{k-1} + alpha X_0, another constant filter that
                                Section 3.1 ("Limitation") lists as precomputable */
} gnnpre_plan_opts_t;

typedef struct gnnpre_plan gnnpre_plan_t; /* opaque; owns device (and pinned host) memory */

typedef struct {
    int64_t n, nnz, nnz_tilde; /* nnz_tilde = |E|: nnz + n for GCN/GIN (self-loops are edges of E), nnz for SAGE */
    int64_t feat_dim;          /* F rounded up to a multiple of 4 */
    int32_t op;
    int32_t b, c;              /* Eq. 12's block counts in use */
    int64_t slab_width;        /* columns per slab: 4 * ceil(F / (4c)) */
    int64_t B_S, B_X, B_fixed; /* Eq. 12's volumes in bytes: 4*nnz_tilde + 8*(n+1); 4*n*F; 16*n (per-node arrays) */
    int64_t beta_S, beta_X;    /* Eq. 12's coefficients as this library sets them */
    int64_t budget_bytes;
    int64_t device_bytes;      /* device memory the plan holds */
    int64_t host_bytes;        /* pinned host memory the plan holds */
    int64_t num_segments;      /* warp-level edge segments over all blocks */
    int64_t num_row_fixups;    /* rows whose edges span more than one segment */
    int64_t num_scratch_rows;  /* partial-sum rows of scratch memory (slab_width floats each) */
    int32_t segment_edges;
    int32_t structure_mem;     /* gnnpre_mem_t: where the plan's copy of E lives: on the host (streamed block by
                                  block) only if the CSR was given on the host and b > 1 was forced or needed */
} gnnpre_plan_info_t;

/* One edge block E^(l): edges [e_lo, e_hi) of the CSR-ordered edge list of the support. */
typedef struct {
    int64_t e_lo, e_hi;
    int32_t row_lo, row_hi;      /* rows holding edge e_lo and edge e_hi - 1 */
    int32_t first_row_partial;   /* row_lo also has edges in block l-1 */
    int32_t last_row_partial;    /* row_hi also has edges in block l+1 */
} gnnpre_block_info_t;

#define GNNPRE_MAX_HOPS 64

typedef struct {
    float hop_ms[GNNPRE_MAX_HOPS]; /* device time per hop (CUDA events); device-resident runs with stats only */
    float total_ms;
    float segments_ms;             /* device time spent in the segment kernel alone, summed over its launches */
    int64_t h2d_bytes, d2h_bytes;  /* streamed runs */
    int64_t kernel_launches;       /* all kernels this call launched */
    int64_t segments_launches;     /* launches of the segment kernel among them */
    float startup_ms;              /* streamed runs with host outputs: call start until the first output copy begins */
    float drain_ms;                /* ... and from there until the last output copy has ended */
    int32_t schedule;              /* GNNPRE_SCHEDULE_*: how the call was run */
    int32_t upload_slabs;          /* column slabs X travelled in (streamed runs with host X) */
} gnnpre_stats_t;

#define GNNPRE_SCHEDULE_RESIDENT 0 /* everything on the device */
#define GNNPRE_SCHEDULE_SLABS 1    /* Algorithm 1's loops, slab loop outermost: c equal slabs, each through all K hops */
#define GNNPRE_SCHEDULE_PANELS 2   /* whole hop matrices on the device, narrow-first column panels (see gnnpre_propagate) */

/*
 * Degrees D_i = number of nonzeros of row i (Section 2).  `deg_out` (int32[n]) lives in the same
 * memory space as the CSR.  Device data: asynchronous on `stream`.  Host data: the row pointers
 * travel through the GPU and the call returns when deg_out is complete.  Integer, exact.
 */
int gnnpre_degrees(const gnnpre_csr_t* csr, int32_t* deg_out, void* stream);

/*
 * Builds the decomposition plan (Section 3.2): validates the CSR, computes degrees (or takes the
 * caller's `degrees`, int32[n] in the CSR's memory space; NULL = compute), the per-node scale
 * factors of the operator (fp64 arithmetic rounded once to fp32), the edge list E of the support
 * with self-loops inserted at their sorted position, (b, c) from Eq. 12 unless forced, the b
 * balanced contiguous edge blocks  [floor(l|E|/b), floor((l+1)|E|/b))  and the warp-level segment
 * tables.  Synchronous.  The plan is immutable afterwards; free it with gnnpre_plan_destroy.
 * While it runs, the build holds the CSR and some flag arrays on the device besides the plan itself
 * (a host-resident CSR is copied there for the duration): about 2 * B_S transient bytes.
 * Errors: INVALID_ARG (NULLs, bad op, F < 1, b > |E|, c > ceil(F/4)), INVALID_CSR, BUDGET_TOO_SMALL, OOM_*, CUDA, UNSUPPORTED_ARCH.
 */
int gnnpre_build_plan(const gnnpre_csr_t* csr, const int32_t* degrees, const gnnpre_plan_opts_t* opts,
                      gnnpre_plan_t** plan_out);

int gnnpre_plan_info(const gnnpre_plan_t* plan, gnnpre_plan_info_t* info_out);

/* Block l in [0, b).  INVALID_ARG outside that range. */
int gnnpre_plan_block(const gnnpre_plan_t* plan, int32_t l, gnnpre_block_info_t* block_out);

/* Host copies for parity checks: degrees int32[n], scales fp32[n] each (A^_ij = rscale_i * cscale_j,
 * times 1 + eps on the GIN diagonal).  Any pointer may be NULL. */
int gnnpre_plan_scales(const gnnpre_plan_t* plan, int32_t* deg_out, float* rscale_out, float* cscale_out);

/* Host copy of the support's CSR: rowptr_out int64[n+1], colidx_out int32[nnz_tilde].  Either may be NULL. */
int gnnpre_plan_support(const gnnpre_plan_t* plan, int64_t* rowptr_out, int32_t* colidx_out);

/*
 * Algorithm 1: out[k-1] <- A^ applied k times to X, for k = 1..K (X itself is not repeated); with a
 * teleport term in the plan, out[k-1] <- (1 - alpha) A^ out[k-2] + alpha X instead.
 *   X      fp32 row-major [n, F] with leading dimension ldx (floats), in x_mem
 *   out    host array of K pointers, each fp32 row-major [n, F] with leading dimension ldo, in out_mem
 *   ldx, ldo >= F rounded up to a multiple of 4 (else INVALID_ARG), themselves multiples of 4, and all base
 *   pointers 16-byte aligned (else GNNPRE_ERR_ALIGN)
 *   out[k] must not overlap X or another out[]; 1 <= K <= GNNPRE_MAX_HOPS
 * Device X and device out: the work is enqueued on `stream` and the call returns at once; the
 * plan's scratch memory is in use until that work completes, so calls on one plan must not
 * overlap on the GPU (use one stream per plan).
 * Any host operand: column slabs of X travel host->device, finished output rows travel
 * device->host on side streams while later blocks compute, and the call returns when out[] is
 * complete in host memory (GNNPRE_ERR_BUSY if another streamed call holds the plan).  Host buffers
 * should be page-locked for full link speed.
 * Host X and host out[] together are run in one of two ways.  If the plan's budget has room for K + 1
 * whole [n, F] matrices besides the plan, c was not forced, F >= 128 is a multiple of 32 and every host
 * row starts on a 128-byte boundary, the hop matrices stay whole on the device and the columns travel in
 * unequal slabs, narrow first (32, 32, 64, 128, ... columns, none wider than the plan's slab width): the
 * first output rows can leave after 1/4 of the time an equal half of X would need, and later outputs
 * leave in wide pieces (a departure from Algorithm 1's equal split ceil(d/c); every column is an
 * independent product, so no result changes).  Otherwise Algorithm 1's loops run with the slab loop
 * outermost, each of the c equal slabs of Eq. 12 through all K hops.  stats->schedule tells which.
 * Accumulation is fp32 in a fixed order: results are bitwise reproducible from run to run for a
 * given plan, and agree across different (b, c) or segment sizes only to rounding.
 * `stats` may be NULL; when given, device-resident calls synchronise `stream` to read the timers.
 * Resuming: every hop depends on the previous one only, so a run interrupted after hop k continues by
 * calling again with X = out[k-1] and K' = K - k (plain filters; bit-identical to the uninterrupted run).
 * With a teleport term X must be X_0, so a resumed run starts from hop 1.
 */
int gnnpre_propagate(gnnpre_plan_t* plan, const float* X, int64_t ldx, int32_t x_mem, int32_t K, float* const* out,
                     int64_t ldo, int32_t out_mem, void* stream, gnnpre_stats_t* stats);

/*
 * The normalised adjacency itself (Eq. 1), computed block-wise as Eq. 10 states it:
 * vals_out[e] = A^_ij for every edge e = (i, j) of the support, in the CSR order that
 * gnnpre_plan_support returns, nnz_tilde fp32 values.  Each value is evaluated in fp64 from the
 * integer degrees and rounded once.  vals_out lives where vals_mem says.  Device-resident structure and
 * output: one launch on `stream`, asynchronous.  Otherwise the plan's b edge blocks play the role of
 * the paper's `a` passes - block E^(l) travels to the device if it lives on the host, its values travel
 * back if wanted on the host, on the plan's copy streams with two buffers of each kind taking turns, so
 * that the upload of block l+1 and the download of block l-1 overlap the kernel of block l - and the call
 * returns when vals_out is complete (GNNPRE_ERR_BUSY if a streamed call holds the plan).
 * gnnpre_propagate never needs this array.
 */
int gnnpre_normalize(gnnpre_plan_t* plan, float* vals_out, int32_t vals_mem, void* stream);

/* Eq. 11 on its own: least a with ceil((alpha_A B_A + alpha_S B_S) / a) + alpha_D B_D <= B_GPU, 1 <= a <= max_a;
 * BUDGET_TOO_SMALL if there is none.  Host only. */
int gnnpre_solve_normalisation_blocks(int64_t B_A, int64_t B_S, int64_t B_D, int64_t alpha_A, int64_t alpha_S,
                                      int64_t alpha_D, int64_t B_GPU, int64_t max_a, int64_t* a_out);

/*
 * Whether a kernel of this plan gave up a wait (no counterpart in the paper).  The bulk-copy kernel never
 * waits without a limit: a wait that runs out sets an error word in the plan, the warp leaves, and the rows
 * it was working on are not valid.  Calls that synchronise anyway (streamed operands, or `stats` given)
 * read that word themselves and return GNNPRE_ERR_TIMEOUT.  A device-resident call without `stats` only
 * enqueues work and returns before it runs, so its caller asks here: this call synchronises `stream` (the
 * stream the work was enqueued on), then returns GNNPRE_ERR_TIMEOUT if the word was set since it was last
 * read, and clears it; GNNPRE_OK otherwise.  Call it after the last gnnpre_propagate /
 * gnnpre_propagate_weighted of a batch, before trusting out[].
 */
int gnnpre_plan_status(gnnpre_plan_t* plan, void* stream);

/*
 * Failure-detection self-test (no counterpart in the paper).  Exercises the give-up path described above
 * without any fault: one warp waits `polls` times (1..100000, each poll parks the warp for up to 20 us) on
 * a barrier that nothing completes, then sets the plan's error word and leaves.
 *   gnnpre_selftest_wait_timeout_async  only enqueues that kernel on `stream`: the caller then sees
 *                                       GNNPRE_ERR_TIMEOUT exactly once through gnnpre_plan_status
 *   gnnpre_selftest_wait_timeout        enqueues it, synchronises and reads the word itself: returns
 *                                       GNNPRE_ERR_TIMEOUT when the path works
 * Either way the device and the plan stay fully usable.
 */
int gnnpre_selftest_wait_timeout_async(gnnpre_plan_t* plan, uint32_t polls, void* stream);
int gnnpre_selftest_wait_timeout(gnnpre_plan_t* plan, uint32_t polls, void* stream);

/*
 * Failure injection for tests (no counterpart in the paper; nothing on the device is made to fail).  After
 * this call the library's next `device_countdown` device allocations succeed and the one after them is
 * reported as failed (GNNPRE_ERR_OOM_DEVICE) without calling the allocator; likewise `host_countdown`
 * for page-locked host allocations (GNNPRE_ERR_OOM_HOST).  One failure per arming; a negative value
 * disarms.  Process-wide.  A call that fails this way must leave no memory behind: gnnpre_build_plan
 * returns *plan_out = NULL, a streamed gnnpre_propagate leaves the plan usable for the next call.
 */
int gnnpre_inject_alloc_failure(int64_t device_countdown, int64_t host_countdown);

/* Waits for the plan's own streams and for the last device-resident call that used it (not for the whole
 * device), then frees everything the plan owns. */
void gnnpre_plan_destroy(gnnpre_plan_t* plan);

/*
 * One hop without any allocation:  out <- A^ X  computed directly from the caller's CSR.
 * (The paper has no counterpart of this call; it exists for callers that must not allocate.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a framework whose memory
 * pool owns the whole device, in a latency-critical loop where an allocation would synchronise the
 * device, or after start-up in a process that has promised a fixed memory footprint.  Such callers
 * cannot use gnnpre_build_plan (it allocates the plan's tables and scratch), so this call takes no
 * plan: it finds rows by searching `rowptr`, recomputes the scale factors on the fly, and keeps the
 * partial sums of rows cut by its segment boundaries in a fixed array of
 * GNNPRE_STATIC_SCRATCH_BYTES bytes that is part of the library's device image (every device that
 * loads the library holds it until the process exits).  It is slower than a planned hop and meant
 * for modest sizes.
 *
 *   csr        device-resident, same contract as gnnpre_csr_t above; NOT validated here
 *   X, out     device, fp32 row-major [n, feat_dim] with leading dimensions ldx, ldo (multiples of 4,
 *              16-byte aligned bases, out != X); feat_dim a multiple of 4, at most 512
 * The work is enqueued on `stream`; the call returns at once and calls no cudaMalloc, cudaFree or
 * other allocating routine.
 * First call on a device: it looks up the device address of the fixed array (once per device, with
 * that device current).  With the driver's default lazy module loading that look-up is also the
 * moment the part of the library that holds the array is loaded onto the device, i.e. when its
 * GNNPRE_STATIC_SCRATCH_BYTES are reserved; if the device has no room left (a memory pool already
 * owns all of it) that first call returns GNNPRE_ERR_OOM_DEVICE or GNNPRE_ERR_CUDA.  So make the first
 * call at start-up, before the process freezes its footprint and outside any stream capture; later
 * calls reserve nothing.  The address is cached per device for the life of the process and does not
 * survive cudaDeviceReset: do not call this function again after resetting a device.
 * Limits: feat_dim <= 512 and 2 * ceil(nnz / 2^20) * feat_dim * 4 <= GNNPRE_STATIC_SCRATCH_BYTES,
 * else GNNPRE_ERR_TOO_LARGE (nothing is launched).
 * All calls on a device share the one array.  Each call overwrites the entries it later reads, so
 * nothing needs clearing between calls, but two calls whose kernels overlap on the GPU (different
 * streams, or different threads) race on it: run them one after the other.
 * Results agree with gnnpre_propagate to rounding (the self-loop term is added last instead of at
 * its sorted position), not bit for bit.
 */
#define GNNPRE_STATIC_SCRATCH_BYTES (64u << 20)
int gnnpre_hop_static(const gnnpre_csr_t* csr, int32_t op, float gin_eps, int64_t feat_dim, const float* X,
                      int64_t ldx, float* out, int64_t ldo, void* stream);

/*
 * K hops as in gnnpre_propagate plus their fixed-weight sum
 *
 *     Z = gamma[0] * X_0 + sum_{k=1..K} gamma[k] * X_k ,      X_k = A^ X_{k-1}  (or the plan's teleport recurrence),
 *
 * i.e. the generalised-PageRank filter of the appendix on GPRGNN (Eq. 13) with weights fixed before training,
 * one of the constant filters Section 3.1 "Limitation" allows to precompute.  Z is accumulated in the epilogue
 * of the kernels that store a finished row, hop by hop (A^^k is never formed), in fp32.
 *
 *   plan       a plan whose structure lives on the device; X, out[], Z are DEVICE pointers (no streamed mode)
 *   gamma      HOST, K + 1 weights
 *   out        HOST array of K device pointers, as in gnnpre_propagate; when only Z is wanted two buffers can
 *              alternate (out[k] == out[k-2] is allowed, out[k] == out[k-1] is not: INVALID_ARG)
 *   Z          device fp32 [n, feat_dim], leading dimension ldz; must not alias X or any out[k]; every element is
 *              overwritten
 * Alignment and leading-dimension rules as for gnnpre_propagate (ldz included).  The work is enqueued on `stream`;
 * the call does not synchronise.
 */
int gnnpre_propagate_weighted(gnnpre_plan_t* plan, const float* X, int64_t ldx, int32_t K, float* const* out, int64_t ldo,
                              const float* gamma, float* Z, int64_t ldz, void* stream);

/*
 * First dense stage of an LC model on a mini-batch of rows (Eq. 9: every term of COMB begins with the
 * k-th precomputed hop times the first weight matrix; the experimental settings use mini-batches of
 * 4096 rows, hidden width 256 and ReLU).  For each hop matrix k < num_hops:
 *
 *     Y_k[i][h] = act_k( sum_f hops[k][batch[i]][f] * Wt[h][f] ),   i < batch_size, h < hidden,
 *
 * act_k = ReLU if bit k of relu_mask is set, else the identity.  The batch rows are gathered by the
 * operand loads of the matrix product; no [batch_size, feat_dim] copy is made.
 *
 *   hops       HOST array of num_hops DEVICE pointers, each fp32 row-major [n, feat_dim] with leading
 *              dimension ldh (the out[] of gnnpre_propagate, or X_0); 1 <= num_hops <= GNNPRE_MAX_HOPS
 *   batch      DEVICE int32[batch_size], row of the hop matrices per output row; NULL = rows
 *              0..batch_size-1 (then batch_size <= n).  NOT validated: an index outside [0, n) reads
 *              as a row of zeros
 *   Wt         DEVICE fp32 [hidden, feat_dim], leading dimension ldw: one row per output unit (the
 *              transpose of Eq. 9's W_1); hidden a multiple of 16, 16 <= hidden <= 256
 *   Y          DEVICE fp32; element (k, i, h) at Y[k * y_hop_stride + i * ldy + h].  y_hop_stride =
 *              batch_size * ldy stacks the hops; y_hop_stride = hidden with ldy = num_hops * hidden
 *              lays them side by side in one row (COMB = concatenation)
 *   error_flag DEVICE int32 or NULL; set to 1 by the kernel if one of its bounded waits ran out
 *              (the results are then invalid).  The caller clears and reads it.
 * ldh, ldw >= feat_dim and ldy >= hidden (else INVALID_ARG); ldh, ldw, ldy, y_hop_stride multiples of 4
 * and all base pointers 16-byte aligned (else ALIGN).  feat_dim itself may be any value >= 1.
 * Arithmetic, by `precision`:
 *   GNNPRE_LC_TF32    tensor cores with tf32 inputs (the low 13 mantissa bits of the fp32 operands are cut,
 *                     not rounded) and fp32 accumulation: |error| <= 2^-9 * sum_f |x||w| plus fp32 summation
 *                     error.  The fastest mode.
 *   GNNPRE_LC_TF32X3  every operand enters as the sum of two tf32 numbers (three tensor-core products per
 *                     term, fp32 accumulation): |error| <= 2^-20 * sum_f |x||w| plus fp32 summation error,
 *                     i.e. fp32-like accuracy.  A CTA then computes at most 128 output columns: with hidden > 128
 *                     the batch rows are fetched twice (the second time mostly from L2) and hidden must be a
 *                     multiple of 64 (else INVALID_ARG).
 * The work is enqueued on `stream` and the call returns without synchronising; nothing is allocated.
 * batch_size = 0 is a no-op.  UNSUPPORTED_ARCH on devices other than compute capability 10.x.
 */
#define GNNPRE_LC_TF32 0
#define GNNPRE_LC_TF32X3 1
int gnnpre_lc_first_layer(const float* const* hops, int32_t num_hops, int64_t n, int64_t feat_dim, int64_t ldh,
                          const int32_t* batch, int64_t batch_size, const float* Wt, int64_t hidden, int64_t ldw,
                          uint64_t relu_mask, int32_t precision, float* Y, int64_t ldy, int64_t y_hop_stride,
                          int32_t* error_flag, void* stream);

/*
 * Failure-detection self-test of gnnpre_lc_first_layer's kernel: one launch (one tile of up to 128 rows of `hop`,
 * tf32 mode) in which the producer warps never announce a chunk, so that every bounded wait of the kernel gives up
 * after `polls` polls (1..100000; a poll parks the warp for at most 20 us).  The kernel must raise the error word,
 * let its copies land, free its tensor memory and return; the call synchronises the stream and returns
 * GNNPRE_ERR_TIMEOUT when the error word was raised (the expected outcome), GNNPRE_OK otherwise.  No wait is
 * unbounded and nothing faults: the device stays usable and a following gnnpre_lc_first_layer call must succeed.
 * Arguments as for gnnpre_lc_first_layer (device pointers; error_flag required; Y receives nothing meaningful).
 */
int gnnpre_lc_selftest_wait_timeout(const float* hop, int64_t n, int64_t feat_dim, int64_t ldh, const float* Wt,
                                    int64_t hidden, int64_t ldw, float* Y, int64_t ldy, int32_t* error_flag,
                                    uint32_t polls, void* stream);

/*
 * Measurement aid (no counterpart in the paper): the fetches of ONE hop and nothing else.  Walks the plan's
 * segments exactly as gnnpre_propagate's segment kernels do - same column tiles, same index stream, same
 * fetch path (128-bit loads into registers, or bulk copies into shared memory, by row width) - adds every
 * fetched row into a plain running sum and writes one float per segment to `sink`.  No scales, no row ends,
 * no compensated sums, no output rows.  Its duration is the yardstick for matrices that fit the L2, where
 * the HBM roofline does not bound a hop: segment-kernel time / this time is the fraction of the device's own
 * gather speed that the kernel reaches.
 *   plan    device-resident structure (else INVALID_ARG)
 *   X       device fp32 [n, F], leading dimension ldx (multiple of 4, base 16-byte aligned)
 *   sink    device fp32 [num_segments] (gnnpre_plan_info); contents meaningless
 * Enqueued on `stream`, asynchronous; the caller times it.  A bounded wait that runs out is reported through
 * gnnpre_plan_status like any other.
 */
int gnnpre_gather_ceiling(gnnpre_plan_t* plan, const float* X, int64_t ldx, float* sink, void* stream);

/*
 * The narrow-first panel schedule of gnnpre_propagate for host X and host out[] (see there), as data: which column
 * slabs X travels in and, in launch order, which hop runs on which columns and which columns of that hop's matrix
 * leave for the host once its edge blocks finish.  Host only, no device needed; exposed so that the schedule's
 * invariants can be checked without a GPU.
 *   feat_dim    F, a multiple of 32;  slab_width  the plan's slab width (>= 64; no slab or job is wider);  K hops
 *   jobs_out    6 int32 per job: hop k (1-based), first column, one past the last column, index of the upload slab
 *               the job waits for (-1: none), first and one-past-last column drained after it (equal: nothing)
 *   max_jobs    capacity of jobs_out in jobs; num_jobs_out receives the real count, num_slabs_out the slab count
 */
int gnnpre_describe_panels(int64_t feat_dim, int64_t slab_width, int32_t K, int32_t* jobs_out, int32_t max_jobs,
                           int32_t* num_slabs_out, int32_t* num_jobs_out);

/* Eq. 12 on its own (exposed for parity with the exhaustive search):
 * least b*c with ceil(beta_S B_S / b) + ceil(beta_X B_X / c) + B_fixed <= B_GPU, 1 <= b <= max_b, 1 <= c <= max_c;
 * ties towards smaller c, then smaller b.  BUDGET_TOO_SMALL if infeasible.  Host only. */
int gnnpre_solve_budget(int64_t B_S, int64_t B_X, int64_t B_fixed, int64_t beta_S, int64_t beta_X, int64_t B_GPU,
                        int64_t max_b, int64_t max_c, int64_t* b_out, int64_t* c_out);

const char* gnnpre_status_string(int status);

/* Text of the last CUDA error this thread saw inside the library ("" if none). */
const char* gnnpre_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* GNNPRE_H */
