/*
 * rubick.h -- C ABI of the B200 (sm_100a) library for the data-parallel hot path of the
 * Rubick scheduler (arXiv 2408.08586): batched evaluation of the paper's training-performance
 * model over every (job x execution plan x resource allocation) candidate, the memory-feasibility
 * mask, the per-(job, allocation) best plan and resource-sensitivity curve, per-job marginal
 * gains, and a greedy allocation round that runs entirely on the device; further the minimum
 * demand of guaranteed jobs and tenant quotas, the incremental round (shrink / exchange step,
 * preemption, reconfiguration gate), batched fitting of the model's coefficients, and a wider plan
 * space (degrees of any size, explicit gradient accumulation).
 *
 * Conventions
 *  - Every call returns an int: RUBICK_OK (0) or a negative error code.  Nothing throws, aborts
 *    or prints.  rubick_last_error(ctx) returns a context-owned, NUL-terminated description of
 *    the last failure on that context.
 *  - Pointer names say where the memory lives: d_ = device memory owned by the CALLER,
 *    h_ = host memory owned by the caller.  The library frees only what it allocated itself
 *    (the context, its tables and scratch).
 *  - All arguments are validated on the host before anything is launched; a rejected call
 *    launches nothing and writes nothing.
 *  - Device work is enqueued on the stream given to rubick_create and is complete after
 *    rubick_sync(ctx) (or the caller's own synchronisation of that stream).  Calls on one
 *    context must not overlap in time from several host threads.
 *  - There is no CPU fallback: without a CUDA device every compute call fails with RUBICK_ECUDA.
 *
 * Index order of the tables (C order, last index fastest):
 *    thr        [J][C][P]      float     predicted samples / second, 0 for an invalid plan
 *    feas       [J][P]         uint32    bit i set <=> plan may run with host-memory level i
 *    best_*     [J][G][C][M]   float / int32
 * with J jobs, P plans, and G / C / M levels of GPUs / CPU cores / host memory.
 */
#ifndef RUBICK_H
#define RUBICK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RUBICK_OK       0
#define RUBICK_EINVAL  (-1)   /* bad argument (sizes, ordering, null pointer, unsupported shape)  */
#define RUBICK_ENOMEM  (-2)   /* a device or host allocation of the library failed                */
#define RUBICK_ECUDA   (-3)   /* the CUDA runtime reported an error (no device, launch failure)   */
#define RUBICK_ESTEPS  (-4)   /* the greedy round stopped at max_steps; the partial result is valid */
#define RUBICK_ESTATE  (-5)   /* call order (no plan space set) or inconsistent table contents    */

#define RUBICK_MAX_G_LEVELS  32
#define RUBICK_MAX_C_LEVELS  64
#define RUBICK_MAX_M_LEVELS  32      /* one feasibility word per (job, plan) */
#define RUBICK_MAX_NODES     4096    /* node state of a round lives in shared memory */
#define RUBICK_MAX_TENANTS   256
#define RUBICK_NOALLOC_MAX_JOBS 32768 /* job limit of rubick_greedy_round_noalloc (1 MiB fixed state) */
#define RUBICK_MAX_PIECES    32      /* nodes a spread job may sit on (gpus_per_node <= 32 for spread placement) */
#define RUBICK_MAX_SPREAD_CLASSES 4

/* per-job status in rubick_assignment */
#define RUBICK_UNALLOCATED 0
#define RUBICK_RUNNING     1
#define RUBICK_PENDING     2         /* guaranteed minimum could not be placed */

/* flags of rubick_best_plan */
#define RUBICK_BEST_RAW    1u        /* per-level best only; default also takes the running maximum over g */

typedef struct rubick_ctx rubick_ctx;

/* Environment (paper Table 1, "Environment" row, plus the node shape of Section 7). */
typedef struct {
    double  B_intra, B_inter, B_pcie;   /* bytes / second inside a node, between nodes, GPU <-> host */
    int64_t gpu_mem_bytes;              /* memory of one GPU                                         */
    int64_t mem_per_node_bytes;         /* host memory of one node                                   */
    int32_t gpus_per_node;              /* must be a power of two                                    */
    int32_t cpus_per_node;
    int32_t bytes_per_elem;             /* 2 = fp16 mixed precision                                  */
    int32_t strict_zero_dp_only;        /* 1: ZeRO stages / offload only for pure data parallelism   */
    int32_t zero3_extra_volume;         /* 0: Section 4.1's V_dp for every ZeRO stage (the paper's rule);
                                           1: stage 3 moves 1.5 x V_dp (parameter gathers on top of the
                                           gradient ring; an option outside the paper)                */
    int32_t reserved;                   /* 0                                                         */
} rubick_env;

/* One job: the model, batch and fitted coefficients of paper Table 1.  Exactly 128 bytes. */
typedef struct {
    double   P;                  /* parameter count (integer-valued)                                */
    int64_t  host_base_bytes;    /* host memory of one training process (one per GPU)               */
    int32_t  l, h, s, b;         /* layers, hidden size, sequence length, global batch              */
    int32_t  mu_cap;             /* largest micro-batch a replica runs at once                      */
    int32_t  alpha_act;          /* activation bytes per (token x hidden unit) per layer            */
    float    tau;                /* forward seconds per sample, whole model on one GPU              */
    float    k_bwd, k_sync, k_opt, k_opt_off, k_off, k_swap, k_const;  /* fittable coefficients     */
    float    w;                  /* weight of this job's throughput in the scheduling objective     */
    int32_t  gmin_idx, cmin_idx; /* guaranteed minimum as level indices; -1 = best effort / none    */
    uint32_t flags;              /* reserved, 0                                                     */
    int32_t  tenant;             /* owner of the job for quota accounting, 0 .. n_tenants - 1       */
    uint8_t  pad[36];
} rubick_job;

/* One execution plan (paper Section 3): DP / TP / PP degrees as log2, ZeRO stage 0..3, gradient
 * checkpointing, ZeRO-Offload; g_level = index of its GPU count 2^(log2d+log2t+log2p) in the grid. */
typedef struct {
    uint8_t log2d, log2t, log2p, zero, gc, off;
    uint8_t g_level;
    uint8_t disabled;            /* non-zero: treat as invalid for every job */
} rubick_plan;

/* One plan of the wider plan space: degrees of any size (the paper's own experiments use a 3-GPU
 * tensor-parallel plan and GPU counts such as 12 and 24).  12 bytes. */
typedef struct {
    uint16_t d, t, p;            /* data / tensor / pipeline parallel degrees, d * t * p = GPUs of the level */
    uint8_t  zero, gc, off;
    uint8_t  g_level;
    uint8_t  disabled;           /* non-zero: treat as invalid for every job */
    uint8_t  accum;              /* explicit gradient accumulation (Table 1's a): the micro-batch is halved this
                                    many times below the largest one a replica may run; 0 = fewest passes */
} rubick_plan_wide;

/* Resource grid: strictly increasing level values on each axis. */
typedef struct {
    int32_t nG, nC, nM;
    int32_t reserved;
    const int32_t *g_levels;         /* GPUs                 [nG] */
    const int32_t *c_levels;         /* CPU cores            [nC] */
    const int64_t *m_levels_bytes;   /* host memory in bytes [nM] */
} rubick_grid;

/* Homogeneous cluster: n_nodes nodes of the environment's shape, all free at the start of a round.
 * Tenant quotas (paper Section 5.1) are optional: with n_tenants > 0, a guaranteed job is placed in
 * the first phase of a round only while its minimum demand (GPUs, cores) fits what is left of its
 * tenant's quota, and uses that much of it once placed; jobs beyond the quota stay PENDING.
 * n_tenants = 0 (pointers ignored): no quotas.  At most RUBICK_MAX_TENANTS tenants. */
typedef struct {
    int32_t n_nodes;
    int32_t n_tenants;
    const int32_t *quota_gpus;       /* host, [n_tenants] */
    const int32_t *quota_cpus;       /* host, [n_tenants] */
} rubick_cluster;

/* Result (and input state) per job. 40 bytes. */
typedef struct {
    int32_t g, c;                /* GPUs and cores held; g == 0: nothing                            */
    int64_t m_bytes;             /* host memory held                                                */
    int32_t plan;                /* plan index, -1 if none                                          */
    int32_t first_node, n_nodes; /* lowest node index used and number of nodes                      */
    float   thr;                 /* predicted throughput of (plan, allocation)                      */
    int32_t status;              /* RUBICK_UNALLOCATED / RUNNING / PENDING                          */
    int32_t m_level;             /* host-memory level index of m_bytes, -1 if none                  */
} rubick_assignment;

/* What a user asked for (paper Section 5.1): resource amounts as level indices and the original
 * plan; plan < 0 marks a best-effort job. 16 bytes. */
typedef struct { int32_t g_idx, c_idx, m_idx, plan; } rubick_request;

/* Per-node state after a round. 24 bytes. */
typedef struct {
    int32_t free_g, free_c;
    int64_t free_m;
    int32_t owner;               /* job that holds this whole node as part of a multi-node set, else -1 */
    int32_t reserved;
} rubick_node;

/* What the reconfiguration gate of an incremental round needs to know about one job slot
 * (paper Section 5.2, "Incorporating reconfiguration penalty"). 16 bytes. */
typedef struct {
    float   T;                   /* seconds the job has trained so far                               */
    float   delta;               /* seconds one checkpoint-resume of the job costs                   */
    int32_t n_reconf;            /* times the job has been reconfigured so far                       */
    int32_t active;              /* 0: the slot is empty (job finished or never submitted)           */
} rubick_reconf;

/* One measured configuration of a model type (Section 4.3): plan index, CPU cores and the throughput
 * observed there; plan < 0 marks an unused slot. 16 bytes. */
typedef struct { int32_t plan; int32_t cores; double thr; } rubick_sample;

#define RUBICK_FIT_PARAMS 7      /* k_bwd, k_sync, k_opt, k_opt_off, k_off, k_swap, k_const (Table 1) */

/* ---- context ---------------------------------------------------------------------------------- */

/* Creates a context bound to CUDA device `device` and to `cuda_stream` (a cudaStream_t passed as
 * void*; NULL = the default stream).  Copies *h_env.  Errors: EINVAL (null pointers, non-positive
 * sizes or bandwidths, gpus_per_node not a power of two), ECUDA (no such device), ENOMEM. */
int rubick_create(rubick_ctx **out, const rubick_env *h_env, int device, void *cuda_stream);

/* Frees the context and everything it allocated.  NULL is allowed. */
void rubick_destroy(rubick_ctx *ctx);

/* Blocks until all work enqueued by this context has finished.  Returns ESTATE if a kernel
 * found inconsistent table contents (a feasibility word that is not a threshold in the level
 * index), ECUDA on a runtime error. */
int rubick_sync(rubick_ctx *ctx);

const char *rubick_last_error(const rubick_ctx *ctx);

/* ---- plan space (host, set-up) ---------------------------------------------------------------- */

/* Enumerates the plan space of Section 3 in canonical order: for every level of h_g_levels that is
 * a power of two, every (d, t, p) of powers of two with d*t*p = g (TP degree ascending, then PP
 * degree ascending), then ZeRO stage 0..3, gradient checkpointing off/on, offload off/on.
 * Writes at most cap plans to h_out, the total count to *n_out (also when it exceeds cap) and, if
 * h_group_off is not NULL, nG + 1 offsets: level i owns plans [off[i], off[i+1]).
 * Pure host code; needs no context and no device. */
int rubick_enumerate_plans(const int32_t *h_g_levels, int nG, rubick_plan *h_out, int cap, int *n_out,
                           int32_t *h_group_off);

/* Installs the plan list and the resource grid (copied; tables are uploaded to the device).
 * Requirements (EINVAL otherwise): 1 <= nG <= RUBICK_MAX_G_LEVELS, 1 <= nC <= RUBICK_MAX_C_LEVELS,
 * 1 <= nM <= RUBICK_MAX_M_LEVELS, strictly increasing positive levels, GPU levels above
 * gpus_per_node multiples of it; P a positive multiple of 4; plans ordered by g_level and laid out
 * in runs of four that share (log2d, log2t, log2p, zero) with (gc, off) = (0,0), (0,1), (1,0), (1,1),
 * and every (d, t, p) with its ZeRO stages 0, 1, 2, 3 in consecutive runs (so P is a multiple of 16),
 * as rubick_enumerate_plans writes them; each plan's GPU count equals g_levels[g_level].  To
 * restrict the space, set `disabled` on plans instead of dropping them. */
int rubick_set_space(rubick_ctx *ctx, const rubick_plan *h_plans, int P, const rubick_grid *h_grid);

/* ---- the hot path ----------------------------------------------------------------------------- */

/* The wider plan space: for EVERY GPU level g (not only powers of two) every ordered factorisation
 * g = d * t * p, in the same canonical order (TP ascending over the divisors of g, then PP, then
 * n_accum accumulation settings 0 .. n_accum - 1, then ZeRO stage, gradient checkpointing,
 * offload); with n_accum = 1 on power-of-two levels the list equals rubick_enumerate_plans'.
 * A plan whose halved micro-batch would hold less than one sample is invalid for that job.
 * Same calling convention; 1 <= n_accum <= 8. */
int rubick_enumerate_plans_wide(const int32_t *h_g_levels, int nG, int n_accum, rubick_plan_wide *h_out, int cap,
                                int *n_out, int32_t *h_group_off);

/* rubick_set_space for plans with degrees of any size.  The evaluation kernels then divide where
 * the power-of-two space shifts (same model, same memory rule, same tolerances); everything
 * downstream (best plan, curves, gains, rounds, fitting) is unchanged.  GPU levels above a node
 * must still be whole nodes. */
int rubick_set_space_wide(rubick_ctx *ctx, const rubick_plan_wide *h_plans, int P, const rubick_grid *h_grid);

/* Candidate table (paper Section 4, Eq. 1 with all its terms; THROUGHPUT = b / T_iter) and the
 * memory-feasibility mask, for jobs d_jobs[0..J).  d_thr: J*C*P floats, d_feas: J*P words, both
 * 16-byte aligned.  To stream a large job set in tiles, call once per tile with offset pointers.
 * J == 0 is allowed and does nothing.  Single-precision arithmetic; masks in exact 64-bit integers. */
int rubick_eval_candidates(rubick_ctx *ctx, const rubick_job *d_jobs, int J, float *d_thr, uint32_t *d_feas);

/* Best plan per (job, GPU level, core level, memory level): the largest d_thr among the level's
 * plans whose feasibility bit is set, lowest plan index on ties, (0, -1, 0) when there is none
 * (Section 5.2: invalid GPU counts have zero throughput).  Unless RUBICK_BEST_RAW is given the
 * result is turned into the resource-sensitivity curve: the running maximum along the GPU axis,
 * carrying the plan and the GPU count actually used (Section 5.2, Fig. 6).
 * d_best_val / d_best_plan / d_best_g: J*G*C*M entries each.  d_thr and d_feas must be 16-byte
 * aligned; table entries must be finite and >= 0 (what rubick_eval_candidates writes).
 * Feasibility words must be thresholds (bit i set implies every higher level bit set); a
 * violation is reported by rubick_sync as ESTATE.  Masks in which the feasible plans of one GPU
 * level share one first level per offload class (all masks of rubick_eval_candidates) take the
 * streaming kernel; any other threshold mask is handled by a slower general kernel with the
 * same results.  The context keeps J + 1 words of scratch (grown on demand with cudaMalloc). */
int rubick_best_plan(rubick_ctx *ctx, const float *d_thr, const uint32_t *d_feas, int J, unsigned flags,
                     float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g);

/* rubick_eval_candidates followed by rubick_best_plan in one pass that never writes the candidate
 * table: the mask (d_feas, J*P words) and the curves (d_best_*, J*G*C*M entries each) are bit-identical
 * to what the two calls produce; only the J*C*P throughputs are not kept.  For callers that want the
 * curves alone (a scheduling round): about 8 bytes per candidate of memory traffic less.
 * d_jobs and d_feas 16-byte aligned; flags as rubick_best_plan. */
int rubick_curves(rubick_ctx *ctx, const rubick_job *d_jobs, int J, unsigned flags, uint32_t *d_feas,
                  float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g);

/* Marginal gain ("slope", Section 5.2) of the next GPU and the next CPU increment of every job in
 * state d_state (fields g, c, thr are read; g == 0 means nothing held): the weighted curve gain
 * per added GPU up to the smallest level that strictly improves on the present value, and per
 * added core up to the next core level, both at the top host-memory level.  d_next_g / d_next_c
 * receive the target level indices (-1 = none), d_gain_* the gains (0 = none). */
int rubick_marginal_gain(rubick_ctx *ctx, const rubick_job *d_jobs, int J, const float *d_curve_val,
                         const rubick_assignment *d_state,
                         float *d_gain_gpu, float *d_gain_cpu, int32_t *d_next_g, int32_t *d_next_c);

/* Minimum demand of guaranteed jobs (Section 5.2, "Scheduling algorithm design"): the job's
 * guaranteed performance is what its original plan predicts at the requested resources
 * (d_thr[j][c_idx][plan] if the plan uses g_levels[g_idx] GPUs and is feasible at memory level
 * m_idx, else 0); its minimum demand is the lexicographically smallest (GPU level, core level), not
 * above the request in either dimension, whose sensitivity-curve value at memory level m_idx is
 * non-zero and reaches that performance; the request itself if there is none.  Writes the two
 * level indices (the values rubick_job.gmin_idx / cmin_idx take) and the guaranteed performance;
 * (-1, -1, 0) for best-effort jobs and for requests with indices off the grid.
 * d_curve_val must be the running-maximum table of rubick_best_plan (not RUBICK_BEST_RAW). */
int rubick_min_resources(rubick_ctx *ctx, const float *d_thr, const uint32_t *d_feas, const float *d_curve_val, int J,
                         const rubick_request *d_req, int32_t *d_gmin_idx, int32_t *d_cmin_idx, float *d_baseline);

/* One greedy scheduling round (Section 5.2, Algorithm 1 in marginal-gain form) on given curve
 * tables, from an empty cluster, entirely on the device: guaranteed minima first, in job order;
 * then repeatedly the placeable increment with the largest positive GPU gain (CPU gain when no
 * GPU increment is left), lowest job index on ties, committed with the best plan and its host
 * memory for the chosen node(s).  d_out: J assignments.  Optional (NULL to skip): d_node_out,
 * n_nodes entries; d_step_log, max_steps int32 entries (job << 2 | type << 1 | accepted);
 * h_steps, the number of increments tried.  Blocks until the round is done.
 * Returns ESTEPS if max_steps was reached first.  The context keeps the round's working tables in
 * scratch of its own, grown on demand with cudaMalloc and kept for later rounds: about 48 bytes per
 * (job, GPU level, core level) and 60 bytes per job. */
int rubick_greedy_round(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                        const float *d_curve_val, const int32_t *d_curve_plan, const int32_t *d_curve_g,
                        const uint32_t *d_feas, const rubick_cluster *h_cluster, int max_steps,
                        rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                        int32_t *h_steps);

/* Model fitting (Section 4.3, "Continuous model fitting"), for J model types at once: chooses the seven
 * fittable parameters of each d_jobs[j] to minimise the root mean squared logarithmic error
 * sqrt(mean_i (ln(1 + predicted throughput_i) - ln(1 + d_samples[j][i].thr))^2) over its S sample slots.
 * The paper names no optimiser: this is a pattern search (exploratory moves on a geometric grid that
 * halves every second sweep, then pattern moves) started from the coefficients in the job record and
 * kept inside fixed bounds (k_bwd 0.25..16, the three overlap exponents 1..16, k_opt 1e-13..1e-9,
 * k_opt_off 1e-10..1e-6, k_const 1e-4..10); `sweeps` sweeps (14 is a good default; at most 64).
 * Double precision.  d_theta: J * 7 doubles in the order of RUBICK_FIT_PARAMS; d_rmsle: J * 2 doubles,
 * the error before and after.  The job records themselves are not modified.  Plans refer to the
 * plan list of rubick_set_space.  Enqueued on the context's stream; errors: EINVAL, ESTATE, ECUDA. */
int rubick_fit_models(rubick_ctx *ctx, const rubick_job *d_jobs, int J, const rubick_sample *d_samples, int S,
                      int sweeps, double *d_theta, double *d_rmsle);

/* One incremental scheduling round (Section 5.2: Algorithm 1 with its shrink step, and
 * "Incorporating reconfiguration penalty") on given curve tables, started from the allocation an
 * earlier round left.  Job slots keep their index between rounds.
 *  - d_prev / d_prev_nodes: the d_out and d_node_out of the earlier round on the same grid and
 *    cluster (both NULL: an empty cluster).  A slot whose previous status is RUNNING keeps its
 *    GPUs, cores, memory, plan and node(s); to retire a finished job clear its status (or mark the
 *    slot inactive in d_reconf) before the call.
 *  - d_reconf (NULL: every slot active, every job free to change): a running job may be touched in
 *    this round only if T > 0 and (T - (n_reconf + 1) * delta) / T > theta (the paper uses 0.97);
 *    otherwise it keeps its allocation and plan.
 *  - A running, unpinned single-node job can be shrunk: GPUs to the next lower level whose own
 *    plans run, cores by one level, never below its guaranteed minimum (the GPUs the curve uses at
 *    (gmin_idx, cmin_idx), and cmin_idx cores); a best-effort job with no lower level is preempted
 *    (status UNALLOCATED).  Jobs that span whole nodes are not shrunk.
 *  - Queued guaranteed jobs are placed first at their minimum, within what their tenant's quota
 *    leaves after the minima of its running guaranteed jobs: on free resources, else by shrinking
 *    the lowest-slope jobs of the first node where that works.  Then increments are taken by
 *    largest gain as in rubick_greedy_round while any fits free resources; when none does, the
 *    largest-gain increment may take resources from the lowest-slope jobs on its node (a queued
 *    job: the first node where it works) while its gain per unit exceeds their loss per unit.  An
 *    exchange is all or nothing; a job shrunk in a round does not grow again in it.
 * d_step_log entries: job << 3 | by exchange << 2 | type << 1 | accepted.  Returns ESTATE when the
 * previous state does not fit the grid or the cluster (outputs are then not written), ESTEPS if
 * max_steps was reached first.  gpus_per_node must not exceed 32.  Blocks until the round is done. */
int rubick_incremental_round(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                             const float *d_curve_val, const int32_t *d_curve_plan, const int32_t *d_curve_g,
                             const uint32_t *d_feas, const rubick_cluster *h_cluster,
                             const rubick_assignment *d_prev, const rubick_node *d_prev_nodes,
                             const rubick_reconf *d_reconf, float theta, int max_steps,
                             rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                             int32_t *h_steps);

/* One scheduling event with state kept in the context: the incremental round on J job slots whose
 * previous allocation, node states and curve tables stay on the device between calls (Section 5.2:
 * curves are "cached for reuse").  h_jobs: all J records (host); only the slots listed in
 * h_changed[0..n_changed) are uploaded and have their tables recomputed (a new arrival, a refitted
 * model); n_changed < 0: all of them.  h_reconf: J gate / activity records (NULL: all active, gate
 * open); clear `active` of a finished job's slot.  The first call, a call with another J or node
 * count, a call after rubick_set_space or rubick_schedule_round*, or restart != 0 starts from an
 * empty cluster with all tables recomputed.  Outputs (host): J assignments, optionally n_nodes
 * node states and the step count.  Errors as rubick_incremental_round. */
int rubick_incremental_event_host(rubick_ctx *ctx, const rubick_job *h_jobs, int J, const rubick_cluster *h_cluster,
                                  const int32_t *h_changed, int n_changed, const rubick_reconf *h_reconf, float theta,
                                  int restart, int max_steps, rubick_assignment *h_out, rubick_node *h_node_out,
                                  int32_t *h_steps);

/* rubick_greedy_round for callers that cannot allocate device memory when they schedule: a
 * daemon that received a fixed device-memory budget at start-up and shares the GPU with jobs
 * that fill the rest (a late cudaMalloc may fail, and stalls the device while it runs), or a
 * process whose device memory belongs to a framework's caching allocator.  (The paper has no counterpart; this is
 * a convenience of this library.)  Same inputs, outputs, order of decisions and return codes
 * as rubick_greedy_round, without the step log and without tenant quotas (n_tenants must be 0).  It calls no cudaMalloc, cudaFree or other
 * allocating routine: the per-job scan state lives in a fixed 1 MiB array inside the library
 * (32 bytes per job), which every GPU that loads the library holds until the process exits.
 *  - J above RUBICK_NOALLOC_MAX_JOBS is rejected with EINVAL and a message naming the limit.
 *  - The first call on a device looks up the array's device address (one cudaGetSymbolAddress
 *    with that device current) and remembers it for the life of the process; make that first call
 *    before any stream capture.  Two host threads may make their first calls at the same time (they
 *    store the same address).  The address belongs to the device's primary context: do not call this
 *    entry point on a device after a cudaDeviceReset of it.
 *  - All calls of this process on the device, from every rubick context, share the one array (another
 *    process has a copy of its own).  The kernel rewrites the state of all J jobs before reading it,
 *    so contents left by an earlier call do no harm; but two calls whose kernels overlap on the GPU
 *    (different streams, different rubick contexts or host threads) race on it and give undefined
 *    results.  Run them one after another. */
int rubick_greedy_round_noalloc(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                                const float *d_curve_val, const int32_t *d_curve_plan, const int32_t *d_curve_g,
                                const uint32_t *d_feas, const rubick_cluster *h_cluster, int max_steps,
                                rubick_assignment *d_out, rubick_node *d_node_out, int32_t *h_steps);

/* The whole path for one scheduling event: candidate table, mask, curves and greedy round for
 * d_jobs[0..J), with the intermediate tables in context-owned scratch (grown on demand, kept
 * between calls).  Outputs as rubick_greedy_round. */
int rubick_schedule_round(rubick_ctx *ctx, const rubick_job *d_jobs, int J, const rubick_cluster *h_cluster,
                          int max_steps, rubick_assignment *d_out, rubick_node *d_node_out, int32_t *h_steps);

/* Same with HOST buffers: copies h_jobs to the device, runs the round, copies the assignments
 * (and node states, if h_node_out is not NULL) back.  h_jobs / h_out may be pageable or pinned. */
int rubick_schedule_round_host(rubick_ctx *ctx, const rubick_job *h_jobs, int J, const rubick_cluster *h_cluster,
                               int max_steps, rubick_assignment *h_out, rubick_node *h_node_out, int32_t *h_steps);

/* ---- spread placement (Section 4.1: groups whose GPUs sit on several nodes communicate at the inter-node
 *      bandwidth; Section 5.2 / Algorithm 1: a job's placement is a list of per-node allocations found node by
 *      node, and the plan is chosen for the placement found) ----------------------------------------------- */

/* Placement class of everything evaluated from now on (rubick_eval_candidates, rubick_curves, rubick_fit_models
 * and the calls built on them).  align = 0 (the default after rubick_set_space*): packed -- a job of at most
 * gpus_per_node GPUs on one node, a larger one on whole nodes.  align = a > 0 (a power of two below
 * gpus_per_node): spread over several nodes in pieces of a GPUs.  Only jobs that one node could hold are spread,
 * in at least two pieces (a < g <= gpus_per_node, a divides g); a tensor-parallel group never straddles pieces
 * (t divides a); a data-parallel group stays inside a piece only if d * t divides a, otherwise its ring runs at
 * B_inter; pipeline traffic always runs at B_inter.  Plans that cannot be spread are invalid in the class
 * (throughput 0, empty mask).  Host call; the plan tables on the device are rebuilt.  Errors: ESTATE (no plan
 * space), EINVAL, ENOMEM, ECUDA. */
int rubick_set_placement(rubick_ctx *ctx, int align);

/* The tables of one spread class, as rubick_curves (or rubick_eval_candidates + rubick_best_plan) wrote them while
 * rubick_set_placement(ctx, align) was in force.  Device pointers, J * G * C * M entries / J * P words. */
typedef struct {
    const float *d_curve_val; const int32_t *d_curve_plan; const int32_t *d_curve_g; const uint32_t *d_feas;
    int32_t align;
    int32_t reserved;
} rubick_spread_class;

/* rubick_greedy_round with spread placement.  The packed tables drive the round as before.  When no node takes a
 * job of at most gpus_per_node GPUs whole (its own node has no room for the increment and no other node fits
 * it), the job is assembled from FREE pieces on several nodes: classes in the order given (widest pieces first),
 * nodes in index order, node n offering min(free GPUs / a, free cores / ceil(c a / g)) pieces, until g / a pieces
 * are found; what the job holds is given back only once the new placement stands.  The commit then takes the
 * highest memory level whose per-piece share ceil(m a / g) fits every node used and reads plan and value from
 * that class's tables; a value that does not improve on the present one rejects the increment as usual.  A job
 * that sits in pieces measures its next increments on its own class's curves; more cores for it stay on its
 * nodes when each has them, otherwise it is placed anew (one node, pieces, or whole nodes from empty ones).
 * d_pieces: J * RUBICK_MAX_PIECES words, node << 8 | GPUs there in ascending node order, -1 = unused;
 * d_class: J words, -1 = packed, k = spread in the k-th class.  For such a job d_out has first_node = its lowest
 * node and n_nodes = the number of nodes used; m_bytes is the plan's memory, shared out evenly over the pieces.
 * n_classes = 0 gives rubick_greedy_round's result.  1 <= gpus_per_node <= 32, no tenant quotas (n_tenants = 0);
 * one single-CTA kernel that rescans every job per step: meant for clusters of a few hundred jobs.
 * The context keeps 32 bytes per job of scratch (grown on demand with cudaMalloc). */
int rubick_greedy_round_spread(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                               const float *d_curve_val, const int32_t *d_curve_plan, const int32_t *d_curve_g,
                               const uint32_t *d_feas, const rubick_spread_class *h_classes, int n_classes,
                               const rubick_cluster *h_cluster, int max_steps, rubick_assignment *d_out,
                               rubick_node *d_node_out, int32_t *d_step_log, int32_t *d_pieces, int32_t *d_class,
                               int32_t *h_steps);

/* ---- measurement aids (the paper has no counterpart) ------------------------------------------- */

#define RUBICK_PROBE_WRITE 0   /* float4 streaming stores over d_buf:            work = bytes written        */
#define RUBICK_PROBE_READ  1   /* float4 streaming loads over d_buf:             work = bytes read           */
#define RUBICK_PROBE_FMA   2   /* single-precision fused multiply-adds in registers: work = FMAs issued      */
#define RUBICK_PROBE_XU    3   /* lg2 / ex2 / rcp approximations in registers:   work = transcendental ops   */

/* Enqueues ONE launch of a machine probe on the context's stream: a micro-kernel that measures the rate
 * roofline fractions are quoted against on this GPU (a write-only and a read-only stream for the table
 * kernels, FP32 and transcendental throughput for the one-pass curves kernel).  The caller times the
 * launch with CUDA events on that stream.  d_buf: device scratch of `bytes` bytes (16-byte aligned, at
 * least 4096; the streams cover all of it, the register probes write at most one word); iters: loop
 * count of the register probes (ignored by the streams).  *h_work (optional) receives the amount of
 * work the launch does, in the unit named above.  Errors: EINVAL, ECUDA. */
int rubick_probe(rubick_ctx *ctx, int kind, void *d_buf, size_t bytes, int iters, double *h_work);

/* Number of kernels this library has launched in this process so far (all contexts; every launch site
 * counts itself).  The difference across a timed region is the number of launches inside it. */
unsigned long long rubick_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* RUBICK_H */
