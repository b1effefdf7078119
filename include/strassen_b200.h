/*
 * strassen_b200 -- C ABI of the single-GPU (NVIDIA B200, sm_100a) hot path of CAPS,
 * the communication-avoiding parallel Strassen algorithm (Ballard, Demmel, Holtz,
 * Lipshitz, Schwartz): the Strassen-Winograd recursion computing C = A.B for n x n
 * FP64 matrices.
 *
 * What one call computes (paper passages in brackets):
 *   - operand formation: the A-side sums T2..T5 and B-side sums S2,S3,S4,S6 of every
 *     live node; the other six operands are plain quadrants and are used in place
 *     [Appendix A; Algorithm 1 "locally compute the S_i's and T_i's"];
 *   - 7^L base-case classical products Q_j = T_j.S_j, one batched FP64 GEMM launch per
 *     group of live leaves [Section 5.4 "switches to classical below some size n0";
 *     Algorithm 2 "localStrassen"];
 *   - recombination of the Q_j into the four quadrants of C through U1..U3
 *     [Appendix A; Algorithm 1 "locally compute C from all the Q_i's"];
 *   - each recursion level runs as a BFS step (all seven sub-problems materialised and
 *     batched) or a DFS step (one sub-problem at a time, its Q_j folded into C and
 *     discarded) [Section 3.1; Algorithm 1], the mix chosen by the workspace budget
 *     with the Limited-Memory rule: the fewest leading DFS steps, then BFS steps only
 *     [Section 3.4];
 *   - odd sizes are handled by dynamic peeling of the last row and column at every
 *     level whose size is odd [Section 3.1 names padding or dynamic peeling].
 *
 * Conventions for every entry point:
 *   - matrices are row-major FP64; "device pointer" means memory the GPU can address
 *     (cudaMalloc or equivalent), "host pointer" ordinary (preferably pinned) host memory;
 *   - functions returning int return STRASSEN_OK (0) or a negative strassen_status;
 *     functions returning a pointer return NULL on failure; either way a description of
 *     the failure is available from strassen_last_error() on the calling thread;
 *   - the library never aborts, throws, or traps on the device; there is no CPU
 *     fallback: without a usable CUDA device the compute calls fail with
 *     STRASSEN_CUDA_ERROR.
 */
#ifndef STRASSEN_B200_H
#define STRASSEN_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct strassen_plan strassen_plan; /* opaque host object */

typedef enum strassen_status {
    STRASSEN_OK = 0,
    STRASSEN_INVALID_ARG = -1,         /* NULL pointer, n < 1, cutoff < 1, batch < 1, ld < n ...       */
    STRASSEN_BAD_SCHEDULE = -2,        /* wrong length or a character other than 'B' / 'D'            */
    STRASSEN_WORKSPACE_TOO_SMALL = -3, /* supplied workspace or budget smaller than the plan needs    */
    STRASSEN_ALIAS = -4,               /* C overlaps A or B                                           */
    STRASSEN_MISALIGNED = -5,          /* a matrix or workspace pointer is not 8-byte (256-byte) aligned */
    STRASSEN_CUDA_ERROR = -6,          /* a CUDA runtime call failed; text in strassen_last_error()   */
    STRASSEN_OUT_OF_MEMORY = -7        /* host or device allocation failed                            */
} strassen_status;

/* Kernel families, used as indices by strassen_plan_get_timings / strassen_plan_launches_of. */
typedef enum strassen_kernel_kind {
    STRASSEN_K_FORM = 0,       /* BFS operand formation: T2..T5, S2,S3,S4,S6 of every parent       */
    STRASSEN_K_GEMM = 1,       /* batched base-case products                                        */
    STRASSEN_K_RECOMBINE = 2,  /* BFS recombination: U-chain, four quadrants of C                   */
    STRASSEN_K_FORM_ONE = 3,   /* DFS operand formation of one sub-problem j                        */
    STRASSEN_K_ACCUMULATE = 4, /* DFS fold of one Q_j into the quadrants of C                       */
    STRASSEN_K_PEEL = 5,       /* peeling fix-ups: rank-one update, last column, last row           */
    STRASSEN_K_SCALE = 6,      /* diagonal scaling passes (STRASSEN_FLAG_SCALE_*)                   */
    STRASSEN_K_FUSED_STEP = 7, /* a whole BFS step of the deepest level (sums, products, U-chain) in one kernel */
    STRASSEN_K_LINCOMB = 8,    /* generic bilinear schemes: linear combinations of blocks / of products       */
    STRASSEN_K_COUNT = 9
} strassen_kernel_kind;

/* Extended plan description.  Zero-initialise, then set what differs from the default. */
typedef struct strassen_options {
    int64_t n;              /* matrix size, >= 1                                                   */
    int64_t cutoff;         /* recurse while the current size is > cutoff; >= 1, or 0 = chosen by the library */
    const char *schedule;   /* one 'B' or 'D' per level, top level first; NULL or "auto" = LM rule */
    int64_t batch;          /* independent products per call; 0 means 1                            */
    int64_t lda, ldb, ldc;  /* leading dimensions in elements; 0 means n                           */
    int64_t stride_a, stride_b, stride_c; /* element distance between batch members; 0 means ld * n */
    size_t workspace_budget_bytes;  /* for "auto": largest workspace allowed; 0 = free device memory
                                       of the current device minus a 1 GiB margin                  */
    int64_t flags;          /* STRASSEN_FLAG_* bits; 0 = defaults                                  */
} strassen_options;

/* By default up to three consecutive BFS levels are formed and recombined in one pass each (the
 * intermediate operands are not read back and the intermediate products never written: fewer HBM
 * bytes, same arithmetic in the same order, bit-identical results).  SINGLE_LEVEL_PASSES keeps one
 * pass per level, TWO_LEVEL_PASSES at most two levels per pass. */
#define STRASSEN_FLAG_SINGLE_LEVEL_PASSES 1
#define STRASSEN_FLAG_TWO_LEVEL_PASSES 32

/* The deepest recursion level, when it is a BFS step, can run as ONE kernel that forms the operand
 * sums in registers while it loads the quadrants of A and B, accumulates the seven products side by
 * side on the FP64 tensor cores and applies the U-chain before it stores C [Section 6.3 "Optimizing
 * on-node performance" asks for such a shared-memory Strassen; Appendix A for the step]: same
 * operations in the same order as the three-launch path, bit-identical results, no workspace traffic
 * for that level.  By default the library uses it where the base products are too few to fill the
 * GPU (small n); FUSED_STEP uses it whenever the deepest level is a BFS step, NO_FUSED_STEP never. */
#define STRASSEN_FLAG_FUSED_STEP 64
#define STRASSEN_FLAG_NO_FUSED_STEP 128

/* A DFS step folds each sub-problem's product Q_j into the quadrants of C [Algorithm 1, "locally compute
 * contribution of Q_i to C"].  Where the sub-problem ends in a one-level recombination pass (a BFS step below
 * it, even size), that pass does the fold itself and Q_j never reaches memory; NO_DFS_FOLD keeps the separate pass
 * (write Q_j, read it back, update C) everywhere.  Same operations on every element either way. */
#define STRASSEN_FLAG_NO_DFS_FOLD 256

/* Replay the plan's launch list as one CUDA graph: the first strassen_dgemm call with a given
 * (A, B, C, workspace) captures the launches on an internal stream and instantiates the graph; that
 * call and every later one with the same pointers costs a single graph launch on the caller's
 * stream (different pointers re-capture).  Meant for launch-bound plans: small n, or DFS-heavy
 * schedules with hundreds of launches.  Per-family timing is not available in this mode (a call
 * made while timing is enabled is enqueued launch by launch). */
#define STRASSEN_FLAG_CUDA_GRAPH 2

/* strassen_dgemm_host only: run consecutive host-buffer products as a pipeline over three streams
 * owned by the plan -- the copy-in of call k+1 beside the products of call k and the copy-out of call
 * k-1 (two sets of device copies; one if the device has no room for two).  `stream` then only waits
 * for this call's result copy: work enqueued on it earlier is NOT waited for, so hostA / hostB must
 * hold their final contents when the call is made, and the host buffers of a call must stay untouched
 * until `stream` (or the device) has been synchronised.  Without this flag everything is enqueued on
 * `stream` in order. */
#define STRASSEN_FLAG_HOST_PIPELINE 4

/* Diagonal scaling for accuracy [Section 6.1: D1 C D3 = (D1 A D2)(D2^-1 B D3)], with power-of-two
 * diagonals so that the scaling itself is exact:
 *   SCALE_OUTSIDE  D1, D3 bring the largest entry of every row of A and of every column of B into
 *                  [1, 2); the error of C_ij then scales with max_k|A_ik| max_k|B_kj| instead of
 *                  max|A| max|B| (the row/column-wise bound of Section 6.1);
 *   SCALE_INSIDE   D2 balances column k of A against row k of B (applied before the outside scaling
 *                  when both are set).
 * Costs three extra passes over A and B, one over C, and 2 n^2 words of workspace (the scaled copies;
 * counted in strassen_plan_workspace_bytes).  A and B themselves are not written. */
#define STRASSEN_FLAG_SCALE_OUTSIDE 8
#define STRASSEN_FLAG_SCALE_INSIDE 16

/*
 * strassen_plan_create -- plan C = A.B for n x n matrices [Algorithm 1 "Require A, B n x n"].
 *   n        matrix size (>= 1), contiguous rows (ld = n), one product per call.
 *   cutoff   base-case size n0 (>= 1): a node of size m is split while m > cutoff, so the
 *            level sizes are m_0 = n, m_{i+1} = floor(m_i / 2); n <= cutoff gives zero
 *            levels, i.e. one classical product [Section 5.4].  0 leaves the number of steps
 *            to the library: with an explicit schedule string it is the string's length; with
 *            NULL / "auto" the steps (base size >= 256) and the interleaving of least estimated
 *            time among all that fit the workspace budget are taken, by the cost model that also
 *            orders strassen_autotune's search [Section 5.4 tunes both by measurement; that is
 *            strassen_autotune].
 *   schedule host string, one character per level from the top: 'B' = BFS step, 'D' = DFS
 *            step [Section 3.1].  NULL or "auto" applies the Limited-Memory rule
 *            [Section 3.4] against the free memory of the current device.
 * Host-only: no device memory is touched until the first strassen_dgemm.  The string is
 * copied.  Returns NULL on failure (see strassen_last_error).
 */
strassen_plan *strassen_plan_create(int64_t n, int64_t cutoff, const char *schedule);

/* strassen_plan_create_ex -- as above with batch, leading dimensions, batch strides and an
 * explicit workspace budget.  `opt` and the string it points to are host memory, read only
 * during the call. */
strassen_plan *strassen_plan_create_ex(const strassen_options *opt);

/*
 * strassen_dgemm -- enqueue C = A.B on `stream` [Algorithm 1; Appendix A].
 *   A, B   device pointers, row-major, n rows of lda / ldb elements (batch members stride_a /
 *          stride_b apart); read only, never written.
 *   C      device pointer, same layout with ldc / stride_c; fully overwritten.  C must not
 *          overlap A or B (checked by address range -> STRASSEN_ALIAS).
 *   stream a cudaStream_t passed as void* (NULL = the legacy default stream).
 * All pointers must be 8-byte aligned (STRASSEN_MISALIGNED otherwise); 16-byte alignment
 * with even leading dimensions selects the vectorised paths.  Asynchronous: returns once
 * the kernels are enqueued; no host synchronisation inside, except on the first call of
 * a plan, which uploads the plan's node tables in `stream` and waits for them (so that later
 * calls may use any other stream) and, unless strassen_plan_set_workspace was called,
 * allocates the workspace (cudaMalloc) -- make that first call outside any stream capture.
 * A plan belongs to the device that was current on its first call (STRASSEN_INVALID_ARG on
 * another one).  One call per plan may be in flight at a time (the workspace is shared).
 * The caller owns A, B, C.  NaN / Inf inputs give unspecified results (the operand sums
 * can turn Inf into NaN where the classical product would not).
 */
int strassen_dgemm(strassen_plan *plan, const double *A, const double *B, double *C, void *stream);

/*
 * strassen_dgemm_host -- the same product for HOST matrices: copies A and B to device
 * staging buffers owned by the plan (allocated on first use), runs strassen_dgemm and
 * copies C back, all enqueued on `stream`; the host buffers must stay valid until the
 * stream has been synchronised.  Host rows are contiguous (ld = n) and batch members n*n
 * apart.  Pinned host memory makes the copies asynchronous.
 */
int strassen_dgemm_host(strassen_plan *plan, const double *hostA, const double *hostB, double *hostC,
                        void *stream);

/* strassen_plan_destroy -- free the plan, its device tables, staging buffers and any
 * workspace it allocated itself (not one given by strassen_plan_set_workspace).  The caller
 * must have synchronised the streams the plan was used on.  NULL is ignored. */
void strassen_plan_destroy(strassen_plan *plan);

/* Bytes of device workspace the resolved schedule needs beyond A, B, C: per BFS level the
 * 4 + 4 operand sums and 7 products of every parent, per DFS level one (T, S, Q) triple per
 * parent, rows padded to a multiple of 4 elements [Sections 3.3.1, 3.4.1: a BFS step stores
 * 7 triples, a DFS step one; the six quadrant operands are used in place here]. */
size_t strassen_plan_workspace_bytes(const strassen_plan *plan);

/* Give the plan caller-owned device memory to use as workspace (256-byte aligned, at least
 * strassen_plan_workspace_bytes).  The plan never frees it.  May be called again between
 * products. */
int strassen_plan_set_workspace(strassen_plan *plan, void *device_ptr, size_t bytes);

/* The resolved schedule string ('B'/'D' per level; "" when there are zero levels).  Owned by
 * the plan. */
const char *strassen_plan_schedule(const strassen_plan *plan);

int strassen_plan_levels(const strassen_plan *plan);                    /* L                         */
int64_t strassen_plan_level_size(const strassen_plan *plan, int level); /* m_level, 0 <= level <= L  */
int64_t strassen_plan_base_size(const strassen_plan *plan);             /* m_L                        */
int64_t strassen_plan_base_products(const strassen_plan *plan);         /* batch * 7^L                */
int64_t strassen_plan_launch_count(const strassen_plan *plan);          /* kernels per strassen_dgemm (counted
                                                                           for a 148-SM device)       */
int64_t strassen_plan_launches_of(const strassen_plan *plan, int kind); /* ... of one family          */

/* Bytes the plan's streaming passes move per product as scheduled: operand formation and recombination
 * of every BFS step (a pass over two or three levels counted with what it really reads and writes, less
 * than one pass per level), formation and fold of every DFS step, the peeled last column and row of
 * odd sizes.  The base products' own operand traffic is not included.  This is the HBM term of the
 * path's roofline [Section 3.3.1 counts the additions of a step; on a GPU they are bound by the bytes]. */
double strassen_plan_pass_bytes(const strassen_plan *plan);

/* The cost model's estimate of one product in milliseconds on a B200 (the estimate that orders
 * strassen_autotune's search and picks plans created with cutoff 0).  Measurement aid. */
double strassen_plan_model_ms(const strassen_plan *plan);

/* Workspace (bytes, unpadded) a schedule string needs under the paper's accounting of 21
 * quarter-size matrices per BFS parent and 3 per DFS parent [Sections 3.3.1, 3.4.1], or,
 * with accounting = 15, counting the six quadrant operands of a BFS step as views.
 * Returns 0 and sets the error text if the arguments are invalid. */
size_t strassen_schedule_model_bytes(int64_t n, int64_t cutoff, int64_t batch, const char *schedule,
                                     int accounting);

/*
 * Per-family device timing [Section 5.2: the paper times the whole product; the split is an
 * addition for roofline reporting].  With timing enabled every launch is bracketed by CUDA
 * events on the call's stream; strassen_plan_get_timings synchronises those events and adds
 * their durations into ms_out[STRASSEN_K_COUNT] (milliseconds since timing was enabled or
 * last read), then clears them.  Off by default.
 */
int strassen_plan_set_timing(strassen_plan *plan, int enabled);
int strassen_plan_get_timings(strassen_plan *plan, double *ms_out /* [STRASSEN_K_COUNT] */);

/*
 * strassen_autotune -- choose the number of Strassen steps and the BFS/DFS interleaving by
 * measurement [Section 5.4: "tuned to use the best interleaving pattern of BFS and DFS steps, and
 * the best total number of Strassen steps"; Section 3.1 on interleaving].
 *
 * Candidates: for every step count L whose base size floor(n / 2^L) is >= min_base, every string of
 * L characters over {B, D} whose workspace fits `workspace_bytes`.  Each candidate runs once to warm
 * up and `repetitions` more times on `stream`, timed with CUDA events; the fastest run counts.  The
 * candidates are tried in the order of a cost model (DMMA time of the base products' tiling + HBM
 * bytes of the passes + launches), most promising first, and the search stops after `max_seconds`.
 * On return *best holds the winner, `log` (if given) the first log_capacity candidates in the order
 * they were tried, and C the product computed with the winner's plan
 * (the stream is synchronised).  A, B, C: device pointers as for strassen_dgemm with ld = n; the
 * caller owns them and the workspace.  Synchronous; allocates only the per-plan node tables.
 */
typedef struct strassen_tune_request {
    int64_t n, batch;          /* batch 0 means 1                                            */
    int64_t min_base;          /* smallest base size considered; 0 means 128                 */
    int repetitions;           /* timed runs per candidate; 0 means 2                        */
    double max_seconds;        /* 0 means 60                                                 */
    const double *A, *B;
    double *C;
    void *workspace;           /* device memory, 256-byte aligned (may be NULL if bytes == 0) */
    size_t workspace_bytes;
    void *stream;
} strassen_tune_request;

typedef struct strassen_tune_entry {
    int64_t cutoff;            /* pass to strassen_plan_create together with schedule        */
    int levels;
    char schedule[36];
    double ms;                 /* best measured time of one product                          */
    double model_ms;           /* the cost model's estimate that ordered the search          */
} strassen_tune_entry;

int strassen_autotune(const strassen_tune_request *request, strassen_tune_entry *best, strassen_tune_entry *log,
                      int log_capacity, int *log_count);

/*
 * Other bilinear schemes through the same traversal [Section 6.6 "Parallelizing other algorithms": every fast
 * square matrix multiplication multiplies n0 x n0 block matrices with q < n0^3 products of linear combinations
 * of the blocks; "the BFS and DFS determine whether the q multiplications are performed in parallel or
 * sequentially"; the recursive classical algorithm is the case q = n0^3].
 *
 * A scheme is three tables of small integers (blocks numbered row-major, b = n0 * block_row + block_column):
 *   u, v   q x n0^2:   T_j = sum_b u[j][b] A_b,   S_j = sum_b v[j][b] B_b,   Q_j = T_j . S_j
 *   w      n0^2 x q:   C_b = sum_j w[b][j] Q_j
 * strassen_scheme_check verifies on the host that the tables multiply matrices (the coefficient of
 * A_(a,b) B_(c,d) in C_(e,f) is 1 where b = c, a = e, d = f and 0 elsewhere); plan creation runs the same check.
 * Built-in names: "classical" (<2,2,2;8>), "strassen" (<2,2,2;7>, the original form with 18 additions),
 * "winograd" (<2,2,2;7>, Appendix A with its shared sub-sums written out).
 *
 * The plan is an ordinary strassen_plan (strassen_dgemm, strassen_dgemm_host, workspace and query calls, destroy).
 * Level rule: m_0 = n, m_{i+1} = m_i / n0 while m_i > cutoff, and every m_i that is split must be divisible by
 * n0 -- generic schemes do not peel (STRASSEN_INVALID_ARG otherwise).  opt->schedule: one 'B' (all q sub-products
 * of a step side by side, batched) or 'D' (one after another, one triple of workspace) per level, or NULL /
 * "auto" for the Limited-Memory rule [Section 3.4].  Combinations that are a single block with coefficient 1 are
 * used in place.  Of opt->flags only CUDA_GRAPH and HOST_PIPELINE apply.  Every linear combination is one
 * streaming launch (each term read once per output element), the products run on the batched FP64 GEMM.
 */
typedef struct strassen_scheme {
    int n0;             /* blocks per side, 2 .. 4                                                   */
    int q;              /* products per step, 1 .. 64                                                */
    const int8_t *u;    /* q x n0^2, row-major, host memory, read during the call only               */
    const int8_t *v;    /* q x n0^2                                                                  */
    const int8_t *w;    /* n0^2 x q                                                                  */
} strassen_scheme;

int strassen_scheme_check(const strassen_scheme *scheme);
strassen_plan *strassen_plan_create_scheme(const strassen_options *opt, const strassen_scheme *scheme);
strassen_plan *strassen_plan_create_named_scheme(const strassen_options *opt, const char *name);

/*
 * The two local steps of ONE BFS step spread over seven GPUs [Algorithm 2, BFS(A, B, C, k) with k = 1:
 * "locally compute T_i, S_i" before the redistribution, "locally compute C from Q_i" after it; Section 3.2 for
 * the layout that makes both communication-free; Section 3.3 for the message size n^2 / (4 P)].  The exchange
 * itself (three all-to-alls among the seven ranks: the T blocks, the S blocks, the Q blocks) is the caller's:
 * the Python layer does it with batched point-to-point operations over NCCL, every block landing in
 * the receiver's own memory before a kernel reads it.
 *
 * Layout.  n even, h = n / 2.  The h rows of every quadrant are cut into seven consecutive blocks of
 * rows_r = floor(h / 7) + (r < h mod 7) rows; rank r owns block r of all four quadrants of A, B and C.  A share
 * is a (2 rows_r) x (2 h) row-major matrix with leading dimension ld >= 2 h: [X11_r | X12_r] above [X21_r | X22_r].
 *
 * strassen_bfs_form_shares: from the rank's shares of A and B, block r of the seven A-side operands T_0..T_6
 * and of the seven B-side operands S_0..S_6 [Appendix A], each rows x h with leading dimension ld_out, written
 * to T_out[j] / S_out[j] (host arrays of seven device pointers): T_out[j] and S_out[j] are what rank r sends to
 * rank j.  Plain quadrants (T_0 = A11, ...) are copied, since they have to travel too.
 *
 * strassen_bfs_combine_shares: from block r of the seven products Q_0..Q_6 (Q_in[j]: rows x h, leading dimension
 * ldq; what rank j sent to rank r), the rank's share of C through the U-chain [Appendix A].
 *
 * Both are asynchronous on `stream`, read every input element once and write every output element once
 * (HBM-bound), never write their inputs, and allocate nothing.  All pointers are device pointers, 8-byte aligned
 * (16-byte alignment with even h and leading dimensions selects 16-byte accesses); rows = 0 is allowed and does
 * nothing.  The sub-product Q_j = T_j . S_j in between is an ordinary strassen_dgemm of size h on rank j.
 */
int strassen_bfs_form_shares(int64_t rows, int64_t h, const double *A_share, int64_t lda, const double *B_share,
                             int64_t ldb, double *const *T_out, double *const *S_out, int64_t ld_out, void *stream);
int strassen_bfs_combine_shares(int64_t rows, int64_t h, const double *const *Q_in, int64_t ldq, double *C_share,
                                int64_t ldc, void *stream);

/*
 * strassen_probe_fp64 -- measure the FP64 arithmetic rate of the current device with a
 * register-resident loop (no memory traffic): kind 0 = scalar fused multiply-add, kind 1..4 =
 * the FP64 tensor-core instruction mma.sync m8n8k4 / m16n8k4 / m16n8k8 / m16n8k16.  Runs
 * `iters` inner iterations per thread on every SM, synchronises, and writes the achieved
 * TFLOP/s to *tflops_out (host pointer).  Measurement aid for the roofline denominator; the
 * paper has no counterpart.
 */
int strassen_probe_fp64(int kind, int64_t iters, void *stream, double *tflops_out);

/*
 * strassen_dgemm_static -- C = A.B for one n x n product, 2 <= n <= STRASSEN_STATIC_MAX_N, WITHOUT
 * allocating anything.  (The paper has no counterpart: this entry point exists for deployment
 * reasons only.)
 *
 * Who it is for: callers that are not allowed to call cudaMalloc / cudaFree when they need a
 * product -- code running under an allocator that has already claimed the whole device and
 * hands out no raw memory, latency-critical loops that cannot afford the device-wide
 * synchronisation an allocation or a free implies, and plug-ins invoked from another library's
 * callback whose contract forbids allocating.  strassen_dgemm cannot serve them: its plan keeps
 * node tables and (unless given one) a workspace in memory it obtains from cudaMalloc.
 *
 * What it computes: exactly one Strassen-Winograd level (a BFS step, with peeling when n is
 * odd) over base products of size floor(n / 2), using the same kernels as strassen_dgemm with
 * cutoff floor(n / 2); the results are identical to that call's.
 *
 * Where the temporaries live: the eight operand sums, the seven products and a small node
 * table (8 entries: the product and its seven sub-products) are kept in a static device array compiled into the library (about 7.9 MB, sized for
 * n = STRASSEN_STATIC_MAX_N).  Every GPU that loads the library holds that array until the
 * process exits.  A larger n is rejected with STRASSEN_WORKSPACE_TOO_SMALL and a message that
 * names the limit; nothing is launched in that case.
 *
 * Arguments: A, B, C device pointers, row-major with contiguous rows (ld = n), 8-byte aligned,
 * C not overlapping A or B; A and B are only read, C is fully overwritten; stream is a
 * cudaStream_t passed as void* (NULL = legacy default stream).  Asynchronous like
 * strassen_dgemm.  Errors are reported the same way (status + strassen_last_error()).
 *
 * Rules that follow from the shared array:
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and the SM count, and sets the
 *     shared-memory attribute of the product kernels (cudaFuncSetAttribute) unless a plan has
 *     done so on that device already; make that first call before starting any stream capture
 *     on that device.  Later calls do no set-up.
 *   - All calls on a device use the same array, and it keeps whatever the previous call left
 *     in it.  No part of it needs to start at zero: every temporary is written in full before
 *     it is read.  Two calls whose kernels can overlap on the GPU (different streams without
 *     an ordering between them, or different host threads doing that) would overwrite each
 *     other's temporaries: order them on one stream or with events.
 *   - The function calls no cudaMalloc, cudaFree, or any routine that allocates device memory.
 */
#define STRASSEN_STATIC_MAX_N 512
int strassen_dgemm_static(int64_t n, const double *A, const double *B, double *C, void *stream);

/* Text describing the last failure on the calling thread ("" if none).  Thread-local. */
const char *strassen_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* STRASSEN_B200_H */
