/*
 * cleave.h -- C ABI of the Cleave hot path on one NVIDIA B200 (sm_100a).
 *
 * The path: every training-step GEMM  C[M x N] = op(A)[M x K] . op(B)[K x N]  is cut into
 * independent sub-GEMM tasks (an output block x a K-slice, shaped by the capabilities of a set of
 * simulated edge devices), all tasks are executed by one persistent grouped-GEMM kernel, the
 * K-split partial blocks are summed in a fixed order into C, and tasks lost to device churn are
 * re-planned over the surviving devices and replayed.
 *
 * Conventions
 *   - Plain C types only.  "host" / "device" on a pointer says where the memory lives.
 *   - All matrices are row-major.  A and B hold bf16 (IEEE binary32 truncated to 16 bits), their
 *     base addresses are 16-byte aligned and their leading dimensions are multiples of 8 elements.
 *   - Every launch is asynchronous on the CUDA stream passed as `void* stream` (a cudaStream_t;
 *     NULL = the legacy default stream).  Nothing synchronises except where stated.
 *   - Return value: 0 on success, a negative CLEAVE_E_* code otherwise.  The library never prints,
 *     throws or exits.  A plan may be used by one host thread at a time.
 *   - There is no CPU fallback and no other backend: without a CUDA device the execution calls
 *     return CLEAVE_E_CUDA.  Planning calls are host-only and work without a device.
 */
#ifndef CLEAVE_H_
#define CLEAVE_H_

#include <stdint.h>

#if defined(__GNUC__)
#define CLEAVE_API __attribute__((visibility("default")))
#else
#define CLEAVE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

/* ---- error codes ------------------------------------------------------------------------- */
#define CLEAVE_OK              0
#define CLEAVE_E_INVAL        -1   /* bad argument (null pointer, zero size, value out of range)   */
#define CLEAVE_E_UNSUPPORTED  -2   /* valid plan or option the kernels cannot run (see the calls)  */
#define CLEAVE_E_INFEASIBLE   -3   /* no plan satisfies the memory constraint                      */
#define CLEAVE_E_NO_DEVICES   -4   /* empty device list, or no surviving device for a GEMM         */
#define CLEAVE_E_RANGE        -5   /* task id >= number of tasks                                   */
#define CLEAVE_E_CUDA         -6   /* a CUDA runtime / driver call failed                          */
#define CLEAVE_E_TIMEOUT      -7   /* a bounded device-side wait expired; the kernel gave up       */
#define CLEAVE_E_BOUNDS       -8   /* a device-side range check failed; the access was skipped     */
#define CLEAVE_E_INCOMPLETE   -9   /* assembly read a block whose task never finished              */
#define CLEAVE_E_NOMEM        -10  /* host or device allocation failed                             */
#define CLEAVE_E_TOOBIG       -11  /* the plan's tables exceed CLEAVE_STATIC_SCRATCH_BYTES         */

/* ---- records ----------------------------------------------------------------------------- */

/* Device record of Section 4.1 ("Communication cost", "Computation cost", "Cost model
 * constraints"): memory capacity M_k [bytes], compute rate F_k [MFLOP/s], downlink / uplink
 * bandwidth W^d_k, W^u_k [bytes/s], downlink / uplink overhead L^d_k, L^u_k [ns].
 * Accepted ranges: mem_bytes <= 2^48, rates and bandwidths in [1, 2^40], latencies <= 2^40. */
typedef struct {
    uint64_t mem_bytes, flops_mflops, dl_Bps, ul_Bps, dl_lat_ns, ul_lat_ns;
} cleave_device_t;

/* One GEMM (Section 4.1, "Search space of GEMM": A_s in R^{m x n}, B_s in R^{n x q}; here
 * M = m_s, K = n_s, N = q_s).
 *   transA = 0: A stored [M x K], lda >= K.   transA = 1: stored [K x M], A[i,k] = X[k,i], lda >= M.
 *   transB = 0: B stored [K x N], ldb >= N.   transB = 1: stored [N x K], B[k,j] = W[j,k], ldb >= K.
 * Forward X.W is (0,0), data gradient dY.W^T is (0,1), weight gradient X^T.dY is (1,0).
 * lda, ldb in elements.  M, N, K < 2^31.
 * level: the GEMM's level in the DAG of the training step (Section 4.1, "Problem definition and
 * objective": GEMMs of one level are independent, a level starts when the level before it has
 * finished).  0 for a flat list.  At most 4096 levels. */
typedef struct {
    uint32_t M, N, K;
    uint32_t lda, ldb;
    uint8_t  transA, transB;
    uint16_t level;
} cleave_gemm_t;

/* One sub-GEMM task: P[alpha x beta] = A[m0:m1, k0:k1] . B[k0:k1, n0:n1]   (alpha = m1-m0 ...).
 * The paper's shard (alpha_{s,p,k}, beta_{s,p,k}) with an added K-range; k0 = 0, k1 = K is the
 * paper's case.  `part_off` is the offset, in fp32 elements, of the task's packed row-major block
 * (leading dimension beta) in the partial arena.  `parent` = id for planned tasks; for a
 * replacement task it is the failed task whose block it rewrites. */
#define CLEAVE_TASK_SUPERSEDED 1u   /* failed and replaced: never executed or waited for again */
#define CLEAVE_TASK_REISSUED   2u   /* created by cleave_reissue                                */
typedef struct {
    uint32_t id, gemm, dev, parent;
    uint32_t m0, m1, n0, n1, k0, k1;
    uint32_t kslice, flags;
    uint64_t part_off;
    uint64_t cost_ns;      /* max(downlink, uplink, compute) on `dev`, Eq. (communication-cost) */
} cleave_task_t;           /* 64 bytes */

/* Planner options.  Zero-initialise and call cleave_plan_opts_default. */
typedef struct {
    uint32_t gran_m, gran_n, gran_k;  /* block granularity in rows / columns / K (128, 128, 128) */
    uint32_t kslice_max;              /* deepest K-slice, 0 = never split for depth (default 4096)*/
    uint32_t ksplit;                  /* 0 = automatic, else the forced number of K-slices        */
    uint32_t ksplit_cap;              /* upper limit of the automatic choice (default 8)          */
    uint32_t reissue_fanout;          /* pieces a failed task is cut into (default 4)             */
    uint32_t b_in, b_out;             /* bytes per input / partial-output element (2, 4)          */
    /* Tail-aware cost (Appendix C, "Tail-Aware Cost Model"): with tail_alpha_milli > 1000 every
     * latency overhead L^d_k, L^u_k is taken as the scale of a Pareto distribution with shape
     * alpha = tail_alpha_milli / 1000 and enters the cost model with its conditional value-at-risk
     * over the worst beta = tail_beta_ppm / 10^6 of outcomes (Eq. 24):
     * L * alpha / ((alpha - 1) * beta^(1/alpha)), rounded up to whole ns.  0 = off (default). */
    uint32_t tail_alpha_milli, tail_beta_ppm;
} cleave_plan_opts_t;

typedef struct cleave_plan_s cleave_plan_t;   /* opaque; owned by the library until cleave_destroy */

/* ---- planning (host only) ---------------------------------------------------------------- */

CLEAVE_API void cleave_plan_opts_default(cleave_plan_opts_t* o);

/* Section 4.1: decide, for every GEMM, the block of rows and columns (and here the K-slice) each
 * device computes, so that the slowest device's max(downlink, uplink, compute) time is small,
 * under exact coverage of the output, the zero-task rule (a device gets a whole block or nothing)
 * and the memory constraint.  Each GEMM is planned independently over the same device list.
 *   g [host, n_gemms], d [host, n_dev], o [host or NULL = defaults]; *out receives the plan.
 * Errors: E_INVAL, E_NO_DEVICES, E_INFEASIBLE, E_NOMEM. */
CLEAVE_API int cleave_plan(const cleave_gemm_t* g, uint32_t n_gemms, const cleave_device_t* d, uint32_t n_dev,
                const cleave_plan_opts_t* o, cleave_plan_t** out);

/* Equal shares (the homogeneous case of Appendix A): rows in grid_m parts, columns in grid_n
 * parts, K in ksplit parts; part sizes floor(x/parts), the first x mod parts one larger.  One
 * implicit device per task (unbounded memory, 1 TFLOP/s, 1 GB/s links, no latency).
 * o may be NULL.  Errors: E_INVAL. */
CLEAVE_API int cleave_plan_uniform(const cleave_gemm_t* g, uint32_t n_gemms, uint32_t grid_m, uint32_t grid_n,
                        uint32_t ksplit, const cleave_plan_opts_t* o, cleave_plan_t** out);

CLEAVE_API uint32_t cleave_plan_num_tasks(const cleave_plan_t* p);        /* planned + reissued             */
CLEAVE_API uint32_t cleave_plan_num_original(const cleave_plan_t* p);     /* planned only                   */
CLEAVE_API const cleave_task_t* cleave_plan_tasks(const cleave_plan_t* p);/* host, id order; valid until the
                                                                  next cleave_reissue / destroy  */
CLEAVE_API uint64_t cleave_plan_arena_elems(const cleave_plan_t* p);      /* fp32 elements of the arena     */
CLEAVE_API uint32_t cleave_plan_ksplit(const cleave_plan_t* p, uint32_t gemm);       /* S of that GEMM      */
CLEAVE_API uint64_t cleave_plan_makespan_ns(const cleave_plan_t* p, uint32_t gemm);  /* modelled, max load  */
CLEAVE_API uint64_t cleave_plan_tstar_ns(const cleave_plan_t* p, uint32_t gemm);     /* water-fill level    */
CLEAVE_API uint32_t cleave_plan_num_tiles(const cleave_plan_t* p);        /* work units of the exec kernel  */
/* Level-wise cost of Section 4.1 (equation "level-cost-s"): the modelled time of a level is that of
 * its slowest GEMM, and levels add up.  cleave_plan_level_makespan_ns: max over the GEMMs of `level`
 * of cleave_plan_makespan_ns (0 for an empty level); cleave_plan_step_makespan_ns: the sum over all
 * levels, the modelled time of the distributed GEMMs of the step. */
/* 1 if the exec kernel can sum the K-slices of this GEMM itself (CLEAVE_EXEC_FINISH), else 0. */
CLEAVE_API uint32_t cleave_plan_finishable(const cleave_plan_t* p, uint32_t gemm);
CLEAVE_API uint32_t cleave_plan_num_levels(const cleave_plan_t* p);
CLEAVE_API uint64_t cleave_plan_level_makespan_ns(const cleave_plan_t* p, uint32_t level);
CLEAVE_API uint64_t cleave_plan_step_makespan_ns(const cleave_plan_t* p);
CLEAVE_API uint32_t cleave_plan_num_launches(const cleave_plan_t* p);     /* kernels launched by one
                                   cleave_exec[_fused] + cleave_assemble, in the current mode    */

/* Host-made failures (Section 3.2, scheduling workflow: a device that leaves is noticed through its
 * broken connection and its unfinished outputs are found in the server's bookkeeping): the
 * listed tasks are skipped by every later cleave_exec / cleave_reissue launch, as if their device
 * had left before returning its block.  Replaces the previous list; n = 0 clears it.
 * ids [host, n].  Errors: E_RANGE. */
CLEAVE_API int cleave_set_drops(cleave_plan_t* p, const uint32_t* ids, uint32_t n);

/* ---- execution (device) ------------------------------------------------------------------ */

/* Runs every live, non-dropped task: P_t = A[m0:m1,k0:k1] . B[k0:k1,n0:n1], bf16 inputs, fp32
 * accumulation, written to partials + part_off (Section 4.1: each device computes
 * A'_{s,p,k} o B'_{s,p,k}, a block of O_s).  Marks each finished task in the plan's bookkeeping.
 *   A, B [host arrays of n_gemms device pointers]; partials [device, >= arena_elems floats,
 *   128-byte aligned].  The first call on a plan creates its device mirrors (allocates).
 * The tensor-core kernel needs: k0 a multiple of 64 and k1 a multiple of 64 or equal to K; m0 a
 * multiple of 8 when transA = 1; n0 a multiple of 8 when transB = 0; lda, ldb multiples of 8.  A
 * plan with a task off these rules (hand-picked granules, ragged uniform grids; the default
 * granules never produce one) is run by a plain CUDA-core kernel instead: same blocks, bookkeeping
 * and churn path, much slower, every block to the arena (the fused calls below then behave as
 * cleave_exec and leave C to cleave_assemble); such a plan must have a single DAG level
 * (else E_UNSUPPORTED).
 * Errors: E_INVAL, E_UNSUPPORTED, E_CUDA, E_NOMEM. */
CLEAVE_API int cleave_exec(cleave_plan_t* p, const void* const* A, const void* const* B, float* partials,
                void* stream);

/* cleave_exec with the write-out of one-slice GEMMs fused into the sub-GEMM kernel.  For a GEMM
 * with a single K-slice a device's block is already a finished block of O (Section 4.1, search
 * space of a GEMM: every device returns a block of the output; the paper's own formulation), so the kernel stores it
 * at its place in C_g instead of the arena and the following cleave_assemble has nothing to do for
 * that GEMM; for GEMMs with several K-slices see CLEAVE_EXEC_FINISH below.  The results are
 * bit-identical to cleave_exec + cleave_assemble.
 *   C [host array of n_gemms device pointers, fp32 row-major, ld = N, 16-byte aligned].  The same C
 *   must be passed to the cleave_assemble that follows; cleave_reissue after a fused execution writes
 *   replacement blocks of one-slice GEMMs to that C as well.  A plain cleave_exec ends fused mode.
 * Errors: as cleave_exec. */
CLEAVE_API int cleave_exec_fused(cleave_plan_t* p, const void* const* A, const void* const* B, float* partials,
                                 float* const* C, void* stream);

/* The general form of the two calls above.  flags (any combination):
 *   CLEAVE_EXEC_DIRECT  blocks of GEMMs with one K-slice are stored at their place in C (as in
 *                       cleave_exec_fused);
 *   CLEAVE_EXEC_FINISH  in a GEMM with several K-slices the block of a cell that is written last
 *                       sums the cell -- every K-slice's block of that cell, read back from the
 *                       arena -- in the fixed tree order of cleave_assemble and stores the sums in C,
 *                       so the server-side aggregation (Section 3.2) needs no pass of its own.  Which
 *                       block comes last changes nothing in the sums: they are bit-identical to
 *                       cleave_assemble's.  Every block is still written to the arena.  GEMMs whose
 *                       K-slices are cut into unequal blocks (after a memory repair), with more than
 *                       8 K-slices or with N % 4 != 0 are left to cleave_assemble; so is every GEMM
 *                       when a task is dropped, and after a cleave_reissue;
 *   CLEAVE_EXEC_CONSUME (with FINISH) the block that completes a cell is used up on arrival: it is
 *                       added to the other K-slices' blocks and never stored in the arena (a third
 *                       less partial-block traffic for two K-slices).  Afterwards the arena holds
 *                       S - 1 of a cell's S blocks, so cleave_verify (E_UNSUPPORTED) and
 *                       cleave_reissue (E_INVAL) are refused until the next execution without it.  Ignored (every block is stored) when a task
 *                       is dropped or superseded, because cleave_assemble will need every block.
 *                       The sums and their bits are the same.
 *   CLEAVE_EXEC_BF16    C holds bf16: every value written to C, by this call and by the
 *                       cleave_assemble / cleave_reissue that follow it, is the fp32 value rounded to
 *                       nearest even (ld = N elements, 16-byte aligned).  Arena blocks stay fp32.
 * cleave_exec_fused is DIRECT | FINISH.  C may be NULL when neither DIRECT nor FINISH is given.
 * level_begin, level_end: only GEMMs with level_begin <= level < level_end run (0, UINT32_MAX: all).
 * Levels run in order inside one launch: a tile of level s starts only after every block of the
 * levels below s (of this launch) has been written, so with DIRECT | FINISH a GEMM may take as A
 * or B what a GEMM of a lower level wrote to its C (bf16) in the same call.  A level that lost a
 * task leaves its output incomplete: after cleave_reissue has replayed it (and cleave_assemble, if
 * the GEMM has several K-slices), run the higher levels again with level_begin.
 * Errors: as cleave_exec. */
#define CLEAVE_EXEC_DIRECT 1u
#define CLEAVE_EXEC_FINISH 2u
#define CLEAVE_EXEC_BF16   4u
#define CLEAVE_EXEC_CONSUME 8u
CLEAVE_API int cleave_exec_opts(cleave_plan_t* p, const void* const* A, const void* const* B, float* partials,
                                void* const* C, uint32_t flags, uint32_t level_begin, uint32_t level_end, void* stream);

/* Parameter-server aggregation (Section 3.1 / 3.2: the server collects the devices' output blocks
 * into the GEMM result; with a K-split collecting means summing): C_g[i,j] = sum over the K-slices s of the partial block covering
 * (i,j) in slice s, as a balanced pairwise tree over adjacent slices padded with +0.0 to a power
 * of two -- a fixed order, so the result is deterministic.
 *   partials [device]; C [host array of n_gemms device pointers], C_g fp32 row-major, ld = N.
 * If a task that feeds C never finished, the device status becomes E_INCOMPLETE (see
 * cleave_status); the sums are still written.  At most 32 K-slices (else E_UNSUPPORTED).
 * What the last execution already wrote to C (see cleave_exec_opts) is not computed again; after an
 * execution with CLEAVE_EXEC_BF16 every C_g holds bf16. */
CLEAVE_API int cleave_assemble(cleave_plan_t* p, const float* partials, float* const* C, void* stream);

/* Churn recovery (Section 4.2): the failed tasks' devices are dead for their GEMM; every failed
 * task is cut by rows into at most reissue_fanout pieces; each piece goes to the surviving device
 * that finishes it earliest under the cache-aware cost (rows / columns a survivor already holds
 * cost no downlink; no downlink latency term), largest piece first; surviving assignments stay
 * fixed.  The pieces are appended to the task list, run like cleave_exec and write into the
 * failed tasks' blocks, so the arena layout and cleave_assemble are unchanged.
 *   failed [host, n].  n = 0: synchronises the stream and takes every live task the bookkeeping
 *   shows unfinished.  Errors: E_RANGE, E_INVAL (already superseded), E_NO_DEVICES, E_INFEASIBLE,
 *   and those of cleave_exec. */
CLEAVE_API int cleave_reissue(cleave_plan_t* p, const uint32_t* failed, uint32_t n,
                   const void* const* A, const void* const* B, float* partials, void* stream);

/* Host-only half of cleave_reissue: appends the replacement tasks for `failed` (same rules, same
 * errors) without launching anything; *first_new receives the id of the first new task.  The new
 * tasks run at the next cleave_exec.  Works without a CUDA device. */
CLEAVE_API int cleave_replan(cleave_plan_t* p, const uint32_t* failed, uint32_t n, uint32_t* first_new);

/* Verification of the returned blocks (Section 6, "Robustness to poisoning attacks": the server
 * dispatched the inputs and received the block, so it can test it with random vectors and
 * matrix-vector products instead of a GEMM).  For every live task t, with vectors r, s of +-1
 * entries,   lhs = r^T P_t s   and   rhs = (A_t^T r) . (B_t s)   are compared:
 * the task is flagged when |lhs - rhs| > tol * (|A_t^T r| . |B_t s|), or when either side is not a
 * number (a block that was never written).  (The paper prints the right side as (A r)^T (B s); with
 * A_t of shape alpha x kappa and r of length alpha it is read as (A_t^T r)^T (B_t s).)
 * Entry e of vector v (0 = r, 1 = s) of task t is -1 when the top bit of SplitMix64's output
 * function applied to seed + (t << 33 | e << 1 | v) is set, else +1.  Sums are fp32: tol = 2e-5
 * accepts honest blocks of the benchmark layers and catches a changed entry larger than about a
 * tenth of a typical one.  Blocks are read from `partials`, or from the C given to the last
 * cleave_exec_fused for one-slice GEMMs.
 *   *n_bad [host] receives the number of flagged tasks.  Synchronises the stream.  The first call
 *   allocates.  Requires K % 4 == 0.  Errors: E_INVAL, E_UNSUPPORTED, E_CUDA, E_NOMEM. */
CLEAVE_API int cleave_verify(cleave_plan_t* p, const void* const* A, const void* const* B, const float* partials,
                             uint64_t seed, float tol, uint32_t* n_bad, void* stream);
/* lhs, rhs, scale, flag (1.0 = flagged) of every task of the last cleave_verify, 4 floats per task,
 * id order; superseded tasks read 0, 0, 0, 0.   out [host, 4 * number of tasks at that call]. */
CLEAVE_API int cleave_verify_values(cleave_plan_t* p, float* out);

/* Synchronises `stream` and returns the device status: 0, E_TIMEOUT or E_BOUNDS (sticky since
 * the last cleave_exec), E_INCOMPLETE (verdict of the latest cleave_assemble), or E_CUDA. */
CLEAVE_API int cleave_status(cleave_plan_t* p, void* stream);

/* Number of finished tiles of each task, copied to host (synchronises the stream).
 * done [host, cleave_plan_num_tasks entries].  A task is finished when the count equals
 * cleave_task_num_tiles. */
CLEAVE_API int cleave_done_counts(cleave_plan_t* p, uint32_t* done, void* stream);
CLEAVE_API uint32_t cleave_task_num_tiles(const cleave_plan_t* p, uint32_t task);

/* Bound, in nanoseconds, of every wait inside the exec kernel (default 2 s).  When a wait runs out
 * the kernel gives up in an orderly way -- its roles leave their loops, tensor-core work in flight
 * is drained, the status becomes E_TIMEOUT -- and the call returns; the plan stays usable.  For
 * tests of that path: with 0 the first wait that is not satisfied at once gives up. */
CLEAVE_API int cleave_set_wait_limit_ns(cleave_plan_t* p, uint64_t ns);

/* Device time of the last exec-kernel and assembly-kernel launches on this plan, in
 * milliseconds, measured with CUDA events on the launching stream (synchronises those events). */
CLEAVE_API int cleave_last_kernel_ms(cleave_plan_t* p, float* exec_ms, float* assemble_ms);

/* cleave_assemble for callers that cannot allocate device memory.  (The paper has no counterpart;
 * this is a convenience of the library.)
 *
 * Some hosts of this library hand all device memory to a pool of their own (a serving process
 * that sizes its caches to the last byte, a framework allocator with a hard memory fraction): a
 * cudaMalloc made behind their back fails or defeats their accounting.  Others sit in a
 * latency-critical loop where cudaMalloc / cudaFree would stall every stream of the device.
 * cleave_assemble allocates its lookup tables on a plan's first use; this variant never calls
 * cudaMalloc, cudaFree or any allocating routine.  Its tables live in a fixed array of
 * CLEAVE_STATIC_SCRATCH_BYTES that belongs to the library image: every device that loads the
 * library holds that much memory until the process exits.
 *
 *   - Same inputs, outputs and arithmetic as cleave_assemble (bit-identical sums); the caller owns
 *     partials and every C[i].  It performs no bookkeeping check: E_INCOMPLETE is never raised, so
 *     use it after a cleave_exec / cleave_reissue that is known to have run every task.
 *   - A plan whose tables do not fit the array is refused with CLEAVE_E_TOOBIG before anything is
 *     launched (about 50 bytes per 16K outputs: the Llama-7B-shaped layer needs ~3 MiB and is
 *     refused, a layer of a quarter of that size fits).
 *   - The first call on each device asks the runtime for the array's address on that device (with
 *     that device current).  Make this first call outside any stream capture.
 *   - All calls share the one array, and it keeps what the last call wrote.  Each call rewrites
 *     every byte its kernels read, in stream order; two calls whose work overlaps on the GPU (on
 *     different streams, or from different threads) race on the array and must be serialised by the
 *     caller.
 * Errors: E_INVAL, E_UNSUPPORTED (more than 32 K-slices), E_TOOBIG, E_CUDA. */
#define CLEAVE_STATIC_SCRATCH_BYTES (2u << 20)
CLEAVE_API int cleave_assemble_static(cleave_plan_t* p, const float* partials, float* const* C, void* stream);

CLEAVE_API void cleave_destroy(cleave_plan_t* p);
CLEAVE_API const char* cleave_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CLEAVE_H_ */
