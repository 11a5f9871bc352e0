/*
 * Rubick oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision CPU statement of what the scheduler's data-parallel
 * path computes: the training-performance model (paper Section 4), the plan space and
 * the best-plan / resource-sensitivity-curve step (Section 5.2), the marginal-gain
 * ("slope") score, one greedy scheduling round (Section 5.2, Algorithm 1, in the
 * grow-only marginal-gain form) and the incremental round with Algorithm 1's shrink step
 * and the reconfiguration gate, plus an exhaustive search used on tiny instances.
 *
 * Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark may
 * build or call this file.  It shares nothing with the CUDA library: no header, no
 * table, no helper.  Inputs arrive as plain arrays of doubles / 64-bit integers, in a
 * layout of its own.
 *
 * Every function is written as the definition it follows, one loop nest per definition,
 * with no blocking, hoisting or caching.
 *
 * Pinning status (see tests/test_oracle_*.py):
 *   - overlap function, communication volumes, pipeline bubble, T_cc, T_opt, T_oo, Eq. 1:
 *     pinned (limits k=1 / k->inf, ring and pipeline simulations, paper-literal special
 *     cases coded separately, homogeneity, monotonicity).
 *   - plan enumeration, best plan, sensitivity curve: pinned (counts, brute force).
 *   - memory-feasibility rule: the paper prints no formula (it defers to the training
 *     frameworks' estimators), so the rule here is this project's reading; it is pinned
 *     only by the three qualitative facts the paper states (Section 2.2, Section 7.2) and
 *     by an independent big-integer recomputation:  "parity unpinned by the paper".
 *   - greedy round: Algorithm 1 is a heuristic with unspecified step sizes; the step list
 *     implemented here is this project's reading; pinned by the exhaustive search
 *     (upper bound, equality on concave single-resource instances) and capacity
 *     invariants, otherwise "parity unpinned by the paper".
 *   - incremental round: same status; pinned by its reductions (empty previous state =
 *     the grow-only round; everything pinned = the previous state), the exhaustive search as
 *     an upper bound, capacity / minimum-demand / gate invariants and hand-made exchanges.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- input layouts (the oracle's own) ------------------------------------------------ */

/* one job = JF_COUNT doubles (integers are stored exactly; all are < 2^53) */
enum {
    JF_P = 0,      /* parameter count (Table 1: P)                       */
    JF_L,          /* layers l                                           */
    JF_H,          /* hidden size h                                      */
    JF_S,          /* sequence length s                                  */
    JF_B,          /* global batch b                                     */
    JF_MUCAP,      /* largest micro-batch one replica may run at once    */
    JF_ALPHA,      /* activation bytes per (token x hidden) per layer    */
    JF_TAU,        /* forward seconds per sample, whole model on one GPU */
    JF_KBWD, JF_KSYNC, JF_KOPT, JF_KOPTOFF, JF_KOFF, JF_KSWAP, JF_KCONST, /* Table 1 fittables */
    JF_W,          /* throughput weight of the job                       */
    JF_GMIN,       /* guaranteed minimum GPU level index, -1 = best effort */
    JF_CMIN,       /* guaranteed minimum CPU level index, -1 = none        */
    JF_HOSTBASE,   /* host bytes per training process (one per GPU)      */
    JF_TENANT,     /* tenant the job belongs to (quota accounting)       */
    JF_COUNT
};

/* environment = EF_COUNT doubles */
enum {
    EF_BINTRA = 0, EF_BINTER, EF_BPCIE, /* bytes / second (Table 1 environment row) */
    EF_GPUMEM,                          /* bytes of memory on one GPU               */
    EF_GN, EF_CN, EF_MN,                /* GPUs, CPU cores, host bytes per node     */
    EF_E,                               /* bytes per element (2 = fp16)             */
    EF_STRICT,                          /* 1: ZeRO / offload only with t = p = 1    */
    EF_Z3VOL,                           /* 1: ZeRO stage 3 moves 1.5 x V_dp (an option outside the paper; 0 = Section 4.1's rule) */
    EF_SPREAD,                          /* placement class of the prediction: 0 = packed (one node, or whole nodes);
                                           a > 0 = spread over several nodes in pieces of a GPUs (Section 4.1: groups
                                           whose GPUs sit on several nodes communicate at the inter-node bandwidth) */
    EF_COUNT
};

/* one plan = 7 int32: d, t, p (degrees themselves), ZeRO stage z, gc, off, and ga = how many times the
 * micro-batch is halved below the largest one a replica may run (explicit gradient accumulation: Table 1
 * lists the accumulation steps a among a plan's parameters; 0 = as few steps as possible) */
enum { PF_D = 0, PF_T, PF_P, PF_Z, PF_GC, PF_OFF, PF_GA, PF_COUNT };

/* terms returned by oracle_terms (for unit tests of the individual formulas) */
enum {
    TF_VALID = 0, TF_MU, TF_M, TF_A,
    TF_TFWD, TF_TBWD,
    TF_VDP, TF_VTP, TF_VPP,
    TF_TDP, TF_TTP, TF_TPP,
    TF_TCC, TF_TOPT, TF_TOFF, TF_TOO, TF_TITER, TF_THR,
    TF_COUNT
};

/* memory terms returned by oracle_memory */
enum {
    MF_PARAMS = 0, MF_GRADS, MF_OPT, MF_ACT, MF_GPU_TOTAL, MF_GPU_OK, MF_HOST_NEED, MF_NODES,
    MF_COUNT
};

/* per-job result of a scheduling round = AF_COUNT int64 + value */
enum { ST_UNALLOCATED = 0, ST_RUNNING = 1, ST_PENDING = 2 };

static int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
static int64_t imin(int64_t a, int64_t b) { return a < b ? a : b; }

/* ---- Section 4.3, "Modeling overlapping": f^k(x, y) = (x^k + y^k)^(1/k) ------------ */
double oracle_overlap(double k, double x, double y)
{
    if (x == 0.0) return y;      /* a zero stage adds nothing (V = 0 rule, Section 4.1) */
    if (y == 0.0) return x;
    return pow(pow(x, k) + pow(y, k), 1.0 / k);
}

/* ---- structural validity of a plan for a job ---------------------------------------- */
static int plan_valid(const double *job, const double *env, const int32_t *pl)
{
    int64_t d = pl[PF_D], t = pl[PF_T], p = pl[PF_P];
    int64_t z = pl[PF_Z], off = pl[PF_OFF];
    int64_t b = (int64_t)job[JF_B], l = (int64_t)job[JF_L], h = (int64_t)job[JF_H];
    int64_t Gn = (int64_t)env[EF_GN];
    if (t > Gn) return 0;                 /* TP stays inside a node (Section 4.1)      */
    if (p > l) return 0;                  /* every stage holds at least one layer      */
    if (d > b || b % d != 0) return 0;    /* at least one whole sample per replica     */
    if (off && z < 2) return 0;           /* offload moves partitioned gradients       */
    if (h % t != 0) return 0;             /* the hidden dimension splits evenly        */
    if (env[EF_STRICT] != 0.0 && (z > 0 || off) && (t > 1 || p > 1)) return 0;
    if (env[EF_SPREAD] != 0.0) {
        /* spread in pieces of a GPUs: only jobs that one node could hold are spread, in at least two pieces,
         * and a tensor-parallel group never straddles two pieces */
        int64_t a = (int64_t)env[EF_SPREAD], g = d * t * p;
        if (g > Gn || g <= a || g % a != 0 || a % t != 0) return 0;
    }
    if (pl[PF_GA] < 0 || pl[PF_GA] > 30) return 0;
    if ((imin(b / d, (int64_t)job[JF_MUCAP]) >> pl[PF_GA]) < 1) return 0;   /* a micro-batch holds at least one sample */
    return 1;
}

/* micro-batching: per-replica batch r = b/d, micro-batch mu = min(r, mu_cap),
 * n = ceil(r / mu) passes.  With pipelining they are the m micro-batches in flight,
 * without it they are the a gradient-accumulation steps (Table 1: m, a). */
static void micro_batching(const double *job, const int32_t *pl, int64_t *mu, int64_t *m, int64_t *a)
{
    int64_t b = (int64_t)job[JF_B], d = pl[PF_D], p = pl[PF_P];
    int64_t r = b / d;
    *mu = imin(r, (int64_t)job[JF_MUCAP]) >> pl[PF_GA];
    int64_t n = cdiv(r, *mu);
    if (p > 1) { *m = n; *a = 1; } else { *m = 1; *a = n; }
}

/* ---- Section 4: all terms of the performance model for (job, plan, c CPU cores) ----- */
void oracle_terms(const double *job, const double *env, const int32_t *pl, double c, double *out)
{
    for (int i = 0; i < TF_COUNT; ++i) out[i] = 0.0;
    if (!plan_valid(job, env, pl)) return;
    out[TF_VALID] = 1.0;

    double d = pl[PF_D], t = pl[PF_T], p = pl[PF_P];
    int z = pl[PF_Z], gc = pl[PF_GC], off = pl[PF_OFF];
    double g = d * t * p;
    double P = job[JF_P], l = job[JF_L], h = job[JF_H], s = job[JF_S], b = job[JF_B];
    double e = env[EF_E], Gn = env[EF_GN];

    int64_t mu_i, m_i, a_i;
    micro_batching(job, pl, &mu_i, &m_i, &a_i);
    double mu = (double)mu_i, m = (double)m_i, a = (double)a_i;
    out[TF_MU] = mu; out[TF_M] = m; out[TF_A] = a;

    /* T_fwd (Section 4.1): forward time of one pass, scaled linearly to the micro-batch
     * and the tensor shard; with pipelining, p stages each holding 1/p of the layers run
     * m + p - 1 slots. */
    double T_fwd = job[JF_TAU] * mu / (t * p);
    if (p > 1) T_fwd *= (m + p - 1.0);
    /* T_bwd = k_bwd * T_fwd, plus one recomputing forward under gradient checkpointing */
    double T_bwd = job[JF_KBWD] * T_fwd + (gc ? T_fwd : 0.0);

    /* volumes in bytes; a degree of 1 sends nothing.  Section 4.1 ("Data Parallelism") gives
     * V_dp = P 2(d-1)/(d t p) and applies it to the whole ZeRO series, so every stage uses it; the
     * environment may switch on a factor 1.5 for stage 3 (parameter gathers on top of the gradient
     * traffic), which is outside the paper and off by default. */
    double V_dp = 0.0, V_tp = 0.0, V_pp = 0.0;
    if (d > 1) V_dp = e * P * 2.0 * (d - 1.0) / (d * t * p) * ((z == 3 && env[EF_Z3VOL] != 0.0) ? 1.5 : 1.0);
    if (t > 1) V_tp = e * 4.0 * 2.0 * (t - 1.0) * b * s * h * l / (d * t);
    if (p > 1) V_pp = e * 2.0 * p * b * s * h / (d * t);

    /* bottleneck bandwidth of each group under the packed placement: ranks are laid out
     * TP fastest, then DP, then PP; g <= Gn sits on one node, larger jobs on whole nodes */
    double B_tp = env[EF_BINTRA];
    double B_dp = (d * t <= Gn) ? env[EF_BINTRA] : env[EF_BINTER];
    double B_pp = (g <= Gn) ? env[EF_BINTRA] : env[EF_BINTER];
    if (env[EF_SPREAD] != 0.0) {
        /* pieces of a GPUs on different nodes: a data-parallel group stays inside a piece only if its d * t
         * consecutive ranks divide the piece; pipeline stages of different pieces talk across nodes */
        double a = env[EF_SPREAD];
        B_dp = fmod(a, d * t) == 0.0 ? env[EF_BINTRA] : env[EF_BINTER];
        B_pp = env[EF_BINTER];
    }
    double T_dp = V_dp / B_dp, T_tp = V_tp / B_tp, T_pp = V_pp / B_pp;

    /* T_cc: a forwards, a-1 plain backwards, the last backward overlapped with the
     * gradient synchronisation, TP / PP traffic on the critical path */
    double T_cc = a * T_fwd + (a - 1.0) * T_bwd
                + oracle_overlap(job[JF_KSYNC], T_bwd, T_dp) + T_tp + T_pp;

    /* optimizer and offloading (Section 4.2) */
    double Psi = P / (t * p);                  /* parameters of one model-parallel shard */
    double T_opt, T_off = 0.0, T_oo;
    if (off) {
        T_opt = job[JF_KOPTOFF] * Psi / (d * c);
        T_off = e * Psi / (d * env[EF_BPCIE]);
        T_oo = oracle_overlap(job[JF_KOFF], T_dp, T_off)
             + oracle_overlap(job[JF_KSWAP], T_opt, T_off);
    } else {
        T_opt = job[JF_KOPT] * Psi / (z >= 1 ? d : 1.0);
        T_oo = T_opt;
    }
    double T_iter = T_cc + T_oo + job[JF_KCONST];      /* Eq. 1 */

    out[TF_TFWD] = T_fwd; out[TF_TBWD] = T_bwd;
    out[TF_VDP] = V_dp; out[TF_VTP] = V_tp; out[TF_VPP] = V_pp;
    out[TF_TDP] = T_dp; out[TF_TTP] = T_tp; out[TF_TPP] = T_pp;
    out[TF_TCC] = T_cc; out[TF_TOPT] = T_opt; out[TF_TOFF] = T_off; out[TF_TOO] = T_oo;
    out[TF_TITER] = T_iter;
    out[TF_THR] = b / T_iter;                           /* THROUGHPUT = b / T_iter */
}

/* ---- memory-feasibility rule (integer bytes) ----------------------------------------- */
void oracle_memory(const double *job, const double *env, const int32_t *pl, int64_t *out)
{
    for (int i = 0; i < MF_COUNT; ++i) out[i] = 0;
    int64_t d = pl[PF_D], t = pl[PF_T], p = pl[PF_P];
    int64_t z = pl[PF_Z], gc = pl[PF_GC], off = pl[PF_OFF];
    int64_t g = d * t * p;
    int64_t Pi = (int64_t)job[JF_P];
    int64_t l = (int64_t)job[JF_L], h = (int64_t)job[JF_H], s = (int64_t)job[JF_S];
    int64_t alpha = (int64_t)job[JF_ALPHA];
    int64_t Gn = (int64_t)env[EF_GN];
    int64_t mu, m, a;
    if (!plan_valid(job, env, pl)) return;
    micro_batching(job, pl, &mu, &m, &a);

    /* model states, mixed-precision Adam: 2 + 2 + 12 bytes per parameter of the shard,
     * ZeRO stage 1 / 2 / 3 spreading optimizer / + gradients / + parameters over d */
    int64_t Psi = cdiv(Pi, t * p);
    int64_t dz1 = z >= 1 ? d : 1, dz2 = z >= 2 ? d : 1, dz3 = z == 3 ? d : 1;
    int64_t params = 2 * cdiv(Psi, dz3);
    int64_t grads = off ? 0 : 2 * cdiv(Psi, dz2);
    int64_t opt = off ? 0 : 12 * cdiv(Psi, dz1);

    /* activations of the layers on one GPU for the micro-batches in flight */
    int64_t A = cdiv(alpha * s * mu * h, t);
    int64_t q = p > 1 ? imin(m, p) : 1;
    int64_t L = cdiv(l, p);
    int64_t act = gc ? L * q * 2 * s * mu * h + A : L * q * A;

    int64_t total = params + grads + opt + act;
    out[MF_PARAMS] = params; out[MF_GRADS] = grads; out[MF_OPT] = opt; out[MF_ACT] = act;
    out[MF_GPU_TOTAL] = total;
    out[MF_GPU_OK] = total <= (int64_t)env[EF_GPUMEM];
    /* host memory: one process per GPU, plus fp32 master weights, momentum, variance and
     * fp16 gradients (4 + 4 + 4 + 2 bytes per parameter) when the optimizer runs on CPUs */
    out[MF_HOST_NEED] = g * (int64_t)job[JF_HOSTBASE] + (off ? 14 * Pi : 0);
    out[MF_NODES] = g <= Gn ? 1 : g / Gn;
}

/* feasibility word: bit i set <=> the plan may run with host-memory level i */
uint32_t oracle_feas_word(const double *job, const double *env, const int32_t *pl,
                          const int64_t *m_levels, int nM)
{
    int64_t mem[MF_COUNT];
    if (!plan_valid(job, env, pl)) return 0u;
    oracle_memory(job, env, pl, mem);
    if (!mem[MF_GPU_OK]) return 0u;
    uint32_t word = 0u;
    for (int i = 0; i < nM; ++i) {
        int ok = mem[MF_HOST_NEED] <= m_levels[i]
              && cdiv(mem[MF_HOST_NEED], mem[MF_NODES]) <= (int64_t)env[EF_MN];
        if (ok) word |= (1u << i);
    }
    return word;
}

/* ---- plan enumeration (Section 3 plan families; canonical order) --------------------- */
static int is_pow2(int64_t x) { return x > 0 && (x & (x - 1)) == 0; }

/* For every GPU level g that is a power of two: all (d, t, p) with d*t*p = g, TP degree
 * ascending, then PP degree ascending, then ZeRO stage, gradient checkpointing, offload.
 * group_off[i] .. group_off[i+1] is the index range of level i.  Returns the plan count
 * (also when it exceeds cap; nothing beyond cap is written). */
int oracle_enumerate_plans(const int64_t *g_levels, int nG, int32_t *plans, int cap, int32_t *group_off)
{
    int n = 0;
    for (int gi = 0; gi < nG; ++gi) {
        group_off[gi] = n;
        int64_t g = g_levels[gi];
        if (!is_pow2(g)) continue;
        for (int64_t t = 1; t <= g; t *= 2)
            for (int64_t p = 1; t * p <= g; p *= 2) {
                int64_t d = g / (t * p);
                for (int z = 0; z < 4; ++z)
                    for (int gc = 0; gc < 2; ++gc)
                        for (int off = 0; off < 2; ++off) {
                            if (n < cap) {
                                int32_t *pl = plans + (size_t)n * PF_COUNT;
                                pl[PF_D] = (int32_t)d; pl[PF_T] = (int32_t)t; pl[PF_P] = (int32_t)p;
                                pl[PF_Z] = z; pl[PF_GC] = gc; pl[PF_OFF] = off; pl[PF_GA] = 0;
                            }
                            ++n;
                        }
            }
    }
    group_off[nG] = n;
    return n;
}

/* The wider plan space of the paper's own experiments (a 3-GPU tensor-parallel plan in Section 7.2,
 * GPU counts such as 12 or 24 in Table 2): for EVERY GPU level g, all ordered factorisations
 * g = d * t * p, TP degree ascending over the divisors of g, then PP degree ascending over the
 * divisors of g / t, then n_ga accumulation settings (the micro-batch halved 0 .. n_ga - 1 times), then
 * ZeRO stage, gradient checkpointing, offload.  With n_ga = 1 on power-of-two levels this is the list of
 * oracle_enumerate_plans. */
int oracle_enumerate_plans_any(const int64_t *g_levels, int nG, int n_ga, int32_t *plans, int cap, int32_t *group_off)
{
    int n = 0;
    for (int gi = 0; gi < nG; ++gi) {
        group_off[gi] = n;
        int64_t g = g_levels[gi];
        for (int64_t t = 1; t <= g; ++t) {
            if (g % t != 0) continue;
            for (int64_t p = 1; p <= g / t; ++p) {
                if ((g / t) % p != 0) continue;
                int64_t d = g / (t * p);
                for (int ga = 0; ga < n_ga; ++ga)
                    for (int z = 0; z < 4; ++z)
                        for (int gc = 0; gc < 2; ++gc)
                            for (int off = 0; off < 2; ++off) {
                                if (n < cap) {
                                    int32_t *pl = plans + (size_t)n * PF_COUNT;
                                    pl[PF_D] = (int32_t)d; pl[PF_T] = (int32_t)t; pl[PF_P] = (int32_t)p;
                                    pl[PF_Z] = z; pl[PF_GC] = gc; pl[PF_OFF] = off; pl[PF_GA] = ga;
                                }
                                ++n;
                            }
            }
        }
    }
    group_off[nG] = n;
    return n;
}

/* ---- candidate table: thr[J][C][P] and feas[J][P] ------------------------------------ */
void oracle_eval(const double *jobs, int J, const int32_t *plans, int P, const double *env,
                 const int64_t *c_levels, int nC, const int64_t *m_levels, int nM,
                 double *thr, uint32_t *feas, int nthreads)
{
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel for schedule(static)
#endif
    for (int j = 0; j < J; ++j) {
        const double *job = jobs + (size_t)j * JF_COUNT;
        double terms[TF_COUNT];
        for (int pi = 0; pi < P; ++pi) {
            const int32_t *pl = plans + (size_t)pi * PF_COUNT;
            for (int ci = 0; ci < nC; ++ci) {
                oracle_terms(job, env, pl, (double)c_levels[ci], terms);
                thr[((size_t)j * nC + ci) * P + pi] = terms[TF_VALID] != 0.0 ? terms[TF_THR] : 0.0;
            }
            feas[(size_t)j * P + pi] = oracle_feas_word(job, env, pl, m_levels, nM);
        }
    }
    (void)nthreads;
}

/* ---- best plan per (job, g level, c level, m level), then the sensitivity curve ------
 * best = the largest predicted throughput among plans using exactly g GPUs that are
 * feasible at host-memory level mi; the lowest plan index wins a tie; (0, -1, 0) if there
 * is none (invalid GPU counts have zero throughput, Fig. 6).  With prefix != 0 the result
 * is the running maximum along g (the curve stays flat over GPU counts that do not
 * improve, Section 5.2), carrying the plan and the GPU count of the earliest maximum. */
void oracle_best_plan(const double *thr, const uint32_t *feas, int J, const int32_t *plans, int P,
                      const int64_t *g_levels, int nG, int nC, int nM, int prefix,
                      double *best_val, int32_t *best_plan, int32_t *best_g, int nthreads)
{
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel for schedule(static)
#endif
    for (int j = 0; j < J; ++j)
        for (int ci = 0; ci < nC; ++ci)
            for (int mi = 0; mi < nM; ++mi) {
                double run_val = 0.0; int32_t run_plan = -1, run_g = 0;
                for (int gi = 0; gi < nG; ++gi) {
                    double bv = 0.0; int32_t bp = -1;
                    for (int pi = 0; pi < P; ++pi) {
                        const int32_t *pl = plans + (size_t)pi * PF_COUNT;
                        int64_t g = (int64_t)pl[PF_D] * pl[PF_T] * pl[PF_P];
                        if (g != g_levels[gi]) continue;
                        if (!((feas[(size_t)j * P + pi] >> mi) & 1u)) continue;
                        double v = thr[((size_t)j * nC + ci) * P + pi];
                        if (v > bv) { bv = v; bp = pi; }
                    }
                    int32_t bg = bp >= 0 ? (int32_t)g_levels[gi] : 0;
                    if (prefix) {
                        if (bv > run_val) { run_val = bv; run_plan = bp; run_g = bg; }
                        bv = run_val; bp = run_plan; bg = run_g;
                    }
                    size_t o = (((size_t)j * nG + gi) * nC + ci) * nM + mi;
                    best_val[o] = bv; best_plan[o] = bp; best_g[o] = bg;
                }
            }
    (void)nthreads;
}

/* ---- minimum demand of a guaranteed job (Section 5.2, "Scheduling algorithm design") --------
 * The job asked for (g_req, c_req, m_req) -- level indices -- with its original plan plan_req.
 * Its guaranteed performance is what that plan predicts there (0 if the plan cannot run there).
 * The minimum demand is the fewest resources, not above the request in any dimension, whose best
 * plan reaches that performance and can run at all (non-zero curve); "fewest" is taken
 * lexicographically, GPUs before cores.  If nothing qualifies the request itself is kept.
 * plan_req < 0 marks a best-effort job: its minimum is nothing (-1, -1).
 * req: [J][4] = g level, c level, m level, plan.  curve: running-maximum table [J][G][C][M]. */
void oracle_min_resources(const double *thr, const uint32_t *feas, const double *curve_val, int J,
                          const int32_t *plans, int P, const int64_t *g_levels, int nG, int nC, int nM,
                          const int64_t *req, int32_t *gmin_idx, int32_t *cmin_idx, double *baseline)
{
    for (int j = 0; j < J; ++j) {
        const int64_t *r = req + (size_t)j * 4;
        int g_req = (int)r[0], c_req = (int)r[1], m_req = (int)r[2], plan = (int)r[3];
        gmin_idx[j] = -1; cmin_idx[j] = -1; baseline[j] = 0.0;
        if (plan < 0) continue;
        double base = 0.0;
        if (plan < P && g_req >= 0 && g_req < nG && c_req >= 0 && c_req < nC && m_req >= 0 && m_req < nM) {
            const int32_t *pl = plans + (size_t)plan * PF_COUNT;
            int64_t g = (int64_t)pl[PF_D] * pl[PF_T] * pl[PF_P];
            if (g == g_levels[g_req] && ((feas[(size_t)j * P + plan] >> m_req) & 1u))
                base = thr[((size_t)j * nC + c_req) * P + plan];
        } else continue;
        baseline[j] = base;
        gmin_idx[j] = g_req; cmin_idx[j] = c_req;
        int found = 0;
        for (int gi = 0; gi <= g_req && !found; ++gi)
            for (int ci = 0; ci <= c_req && !found; ++ci) {
                double v = curve_val[(((size_t)j * nG + gi) * nC + ci) * nM + m_req];
                if (v > 0.0 && v >= base) { gmin_idx[j] = gi; cmin_idx[j] = ci; found = 1; }
            }
    }
}

/* ======================================================================================
 * Scheduling: marginal gains and one greedy round.
 *
 * Two arithmetic forms of the same step list.  The default takes every decision in single
 * precision on a single-precision curve table, with one rounding per operation in the order
 * written (compile with -ffp-contract=off), so that a second implementation can reproduce every
 * comparison bit for bit.  With a double-precision curve table (Sched.cv64) the same decisions
 * are taken in double precision on it; the two forms may part only at a decision whose margin
 * is within the rounding of the single-precision form (tests/test_oracle_sched.py).
 * ==================================================================================== */

typedef struct {
    int J, nG, nC, nM, P, N;
    const float *cv;          /* curve value   [J][G][C][M] */
    const double *cv64;       /* the same table in double precision: decisions in double (NULL: in single on cv) */
    const int32_t *cp;        /* curve plan    [J][G][C][M] */
    const int32_t *cg;        /* curve g used  [J][G][C][M] */
    const uint32_t *feas;     /* [J][P] */
    const double *jobs;
    const int64_t *g_levels, *c_levels, *m_levels;
    int64_t Gn, Cn, Mn;
    /* cluster state */
    int64_t *free_g, *free_c, *free_m;
    int32_t *owner;           /* job holding the whole node as part of a multi-node set, or -1 */
    /* spread placement classes (none: nK = 0): tables predicted for pieces of align[k] GPUs on several nodes */
    int nK;
    const int64_t *align;
    const float *const *kcv; const int32_t *const *kcp; const int32_t *const *kcg; const uint32_t *const *kfeas;
    int *piece_n, *piece_q;   /* [J][MAX_PIECES], only with spread classes */
} Sched;

#define MAX_PIECES 32         /* a spread job sits on at most this many nodes (gpus per node <= 32) */

typedef struct {
    int gi, ci;               /* level indices, gi = -1 when unallocated */
    int64_t g, c, m;          /* amounts held (m in bytes)               */
    int plan, node, k;        /* plan index, first node, node count      */
    double val;               /* predicted throughput of the allocation (a float's value in the single-precision form) */
    int status;
    int frozen[2];            /* a rejected GPU / CPU increment is not retried this round */
    int cls;                  /* -1: packed placement; k >= 0: spread in pieces of align[k] GPUs */
    int np;                   /* spread: number of nodes used; the nodes (ascending) and the pieces on each are in
                                 Sched.piece_n / piece_q [job][MAX_PIECES] */
} JobState;

typedef struct { int ok; int k; int stay; int node; int need_new; int cls; int np; int pn[MAX_PIECES], pq[MAX_PIECES]; } Place;

static size_t cidx(const Sched *S, int j, int gi, int ci, int mi)
{
    return (((size_t)j * S->nG + gi) * S->nC + ci) * S->nM + mi;
}

/* curve value at a table offset, in the precision the decisions are taken in */
static double cval(const Sched *S, size_t o) { return S->cv64 ? S->cv64[o] : (double)S->cv[o]; }
/* the same on the curve of the placement class a job holds (a spread job's next steps are measured on the
 * predictions of its own class, so that an increment is not credited with merely undoing the spreading) */
static double cval_of(const Sched *S, const JobState *js, size_t o)
{
    return (js->gi >= 0 && js->cls >= 0) ? (double)S->kcv[js->cls][o] : cval(S, o);
}

/* weighted gain per unit, (w v - w v_cur) / units, one rounding per operation */
static double unit_gain(const Sched *S, double w, double v, double vcur, double units)
{
    if (S->cv64) return (w * v - w * vcur) / units;
    float wf = (float)w;
    return (double)((wf * (float)v - wf * (float)vcur) / (float)units);
}

static int count_empty(const Sched *S)
{
    int n = 0;
    for (int i = 0; i < S->N; ++i) n += (S->free_g[i] == S->Gn);
    return n;
}

/* Where would job js run with g2 GPUs and c2 cores?  One node if g2 <= Gn: its present
 * node when the increment fits there, else the first node (index order) with room for the
 * whole job.  Otherwise g2 / Gn whole nodes: those it already holds entirely plus the
 * lowest-numbered empty ones, with ceil(c2 / k) cores on each. */
static Place find_place_of(const Sched *S, int j, const JobState *js, int64_t g2, int64_t c2)
{
    const int *jpn = S->piece_n ? S->piece_n + (size_t)j * MAX_PIECES : NULL, *jpq = S->piece_q ? S->piece_q + (size_t)j * MAX_PIECES : NULL;
    Place pl; pl.ok = 0; pl.k = 1; pl.stay = 0; pl.node = -1; pl.need_new = 0; pl.cls = -1; pl.np = 0;
    int allocated = js->gi >= 0;
    int spread = allocated && js->cls >= 0;
    if (g2 <= S->Gn) {
        if (allocated && !spread && js->k == 1
            && S->free_g[js->node] >= g2 - js->g && S->free_c[js->node] >= c2 - js->c) {
            pl.ok = 1; pl.stay = 1; pl.node = js->node; return pl;
        }
        if (spread && g2 == js->g) {
            /* more cores for a spread job: it stays where it is when every node it uses has the extra cores */
            int64_t a = S->align[js->cls];
            int64_t extra = cdiv(c2 * a, g2) - cdiv(js->c * a, js->g);
            int fits = 1;
            for (int i = 0; i < js->np; ++i) if (S->free_c[jpn[i]] < extra * jpq[i]) fits = 0;
            if (fits) {
                pl.ok = 1; pl.stay = 1; pl.cls = js->cls; pl.np = js->np; pl.node = jpn[0];
                for (int i = 0; i < js->np; ++i) { pl.pn[i] = jpn[i]; pl.pq[i] = jpq[i]; }
                return pl;
            }
        }
        for (int n = 0; n < S->N; ++n)
            if (S->free_g[n] >= g2 && S->free_c[n] >= c2) { pl.ok = 1; pl.node = n; return pl; }
        /* No node takes the whole job: assemble it from free pieces on several nodes, in node order, for the
         * first spread class (they come with the widest pieces first) that finds enough of them.  A piece is
         * a GPUs with the job's cores shared out evenly, ceil(c a / g) a piece.  What the job holds now is not
         * counted: it is given back only once the new placement stands. */
        for (int kx = 0; kx < S->nK; ++kx) {
            int64_t a = S->align[kx];
            if (a <= 0 || g2 % a != 0 || g2 <= a) continue;
            int64_t want = g2 / a, cpp = cdiv(c2 * a, g2);
            int np = 0; int64_t left = want;
            for (int n = 0; n < S->N && left > 0 && np < MAX_PIECES; ++n) {
                int64_t q = imin(S->free_g[n] / a, S->free_c[n] / cpp);
                if (q <= 0) continue;
                if (q > left) q = left;
                pl.pn[np] = n; pl.pq[np] = (int)q; ++np; left -= q;
            }
            if (left == 0) { pl.ok = 1; pl.cls = kx; pl.np = np; pl.node = pl.pn[0]; return pl; }
        }
        return pl;
    }
    if (g2 % S->Gn != 0) return pl;
    int k2 = (int)(g2 / S->Gn);
    pl.k = k2;
    if (cdiv(c2, k2) > S->Cn) return pl;
    int empty = count_empty(S);
    if (allocated && !spread && js->g >= S->Gn) {            /* holds whole nodes already */
        if (k2 == js->k) { pl.ok = 1; pl.stay = 1; pl.node = js->node; return pl; }
        pl.need_new = k2 - js->k;
        pl.stay = 1;
    } else {
        pl.need_new = k2;
        if (allocated && !spread && S->free_g[js->node] + js->g == S->Gn) empty += 1; /* its node empties */
    }
    pl.ok = empty >= pl.need_new;
    return pl;
}

static void release_job(Sched *S, int j, JobState *js)
{
    if (js->gi < 0) return;
    if (js->cls >= 0) {
        /* spread: every piece gives back a GPUs and its even share of the cores and of the memory */
        int64_t a = S->align[js->cls];
        int64_t cpp = cdiv(js->c * a, js->g), mpp = cdiv(js->m * a, js->g);
        const int *jpn = S->piece_n + (size_t)j * MAX_PIECES, *jpq = S->piece_q + (size_t)j * MAX_PIECES;
        for (int i = 0; i < js->np; ++i) {
            int n = jpn[i];
            S->free_g[n] += a * jpq[i]; S->free_c[n] += cpp * jpq[i]; S->free_m[n] += mpp * jpq[i];
        }
        return;
    }
    if (js->k == 1) {
        S->free_g[js->node] += js->g; S->free_c[js->node] += js->c; S->free_m[js->node] += js->m;
    } else {
        for (int n = 0; n < S->N; ++n)
            if (S->owner[n] == j) {
                S->free_g[n] += S->Gn; S->free_c[n] += cdiv(js->c, js->k); S->free_m[n] += cdiv(js->m, js->k);
                S->owner[n] = -1;
            }
    }
}

/* highest host-memory level whose per-node share fits the node(s) of placement pl (-1: none) */
static int commit_level(const Sched *S, const JobState *js, Place pl, int64_t g2)
{
    if (pl.cls >= 0) {
        /* spread: a level fits when every node holds the share of its pieces, ceil(m a / g) a piece (a job
         * that stays has its present share of that node on top of what is free) */
        int64_t a = S->align[pl.cls];
        int64_t own = (pl.stay && js->gi >= 0) ? cdiv(js->m * a, js->g) : 0;
        int mi = -1;
        for (int i = 0; i < S->nM; ++i) {
            int64_t mpp = cdiv(S->m_levels[i] * a, g2);
            int fits = 1;
            for (int q = 0; q < pl.np; ++q) if (mpp * pl.pq[q] > S->free_m[pl.pn[q]] + own * pl.pq[q]) fits = 0;
            if (fits) mi = i;
        }
        return mi;
    }
    int k2 = pl.k;
    int64_t avail;
    if (k2 > 1) avail = S->Mn;
    else avail = S->free_m[pl.node] + ((pl.stay && js->gi >= 0) ? js->m : 0);
    int mi = -1;
    for (int i = 0; i < S->nM; ++i)
        if (cdiv(S->m_levels[i], k2) <= avail) mi = i;
    return mi;
}

/* Commit job j to (gi2, ci2) at placement pl: pick the host-memory level that fits the
 * target node(s), read the curve there (GetBestPlan), allocate that plan's memory
 * (AllocMem).  Returns 1 on success; 0 leaves everything unchanged.  need_gain != 0
 * additionally demands a strictly higher value than the job has now. */
static int commit(Sched *S, int j, JobState *js, int gi2, int ci2, Place pl, int need_gain)
{
    int64_t g2 = S->g_levels[gi2], c2 = S->c_levels[ci2];
    int k2 = pl.k;
    int mi = commit_level(S, js, pl, g2);
    if (mi < 0) return 0;
    size_t o = cidx(S, j, gi2, ci2, mi);
    /* GetBestPlan for the placement found: a spread placement reads the tables of its class */
    double v = cval(S, o); int plan = S->cp[o]; int gu = S->cg[o];
    const uint32_t *feas_tab = S->feas;
    if (pl.cls >= 0) { v = (double)S->kcv[pl.cls][o]; plan = S->kcp[pl.cls][o]; gu = S->kcg[pl.cls][o]; feas_tab = S->kfeas[pl.cls]; }
    if (plan < 0 || !(v > 0.0)) return 0;
    if ((int64_t)gu != g2) return 0;              /* the level's own plans do not fit */
    if (need_gain && js->gi >= 0 && !(v > js->val)) return 0;
    uint32_t word = feas_tab[(size_t)j * S->P + plan];
    int f = 0; while (f < S->nM && !((word >> f) & 1u)) ++f;
    if (f > mi) return 0;
    int64_t m2 = S->m_levels[f];

    /* remember whole nodes held, then give everything back and take the new placement */
    int *keep = NULL; int nkeep = 0;
    if (k2 > 1 && pl.stay && js->gi >= 0) {
        keep = (int *)malloc(sizeof(int) * (size_t)S->N);
        if (js->k == 1) keep[nkeep++] = js->node;
        else for (int n = 0; n < S->N; ++n) if (S->owner[n] == j) keep[nkeep++] = n;
    }
    release_job(S, j, js);
    if (pl.cls >= 0) {
        int64_t a = S->align[pl.cls];
        int64_t cpp = cdiv(c2 * a, g2), mpp = cdiv(m2 * a, g2);
        for (int i = 0; i < pl.np; ++i) {
            int n = pl.pn[i];
            S->free_g[n] -= a * pl.pq[i]; S->free_c[n] -= cpp * pl.pq[i]; S->free_m[n] -= mpp * pl.pq[i];
            S->piece_n[(size_t)j * MAX_PIECES + i] = n; S->piece_q[(size_t)j * MAX_PIECES + i] = pl.pq[i];
        }
        js->np = pl.np; js->node = pl.pn[0];
    } else if (k2 == 1) {
        S->free_g[pl.node] -= g2; S->free_c[pl.node] -= c2; S->free_m[pl.node] -= m2;
        js->node = pl.node;
    } else {
        int taken = 0, first = -1;
        int64_t cs = cdiv(c2, k2), ms = cdiv(m2, k2);
        for (int i = 0; i < nkeep; ++i) {
            int n = keep[i];
            S->free_g[n] -= S->Gn; S->free_c[n] -= cs; S->free_m[n] -= ms; S->owner[n] = j; ++taken;
        }
        for (int n = 0; n < S->N && taken < k2; ++n)
            if (S->owner[n] != j && S->free_g[n] == S->Gn) {
                S->free_g[n] -= S->Gn; S->free_c[n] -= cs; S->free_m[n] -= ms; S->owner[n] = j; ++taken;
            }
        for (int n = 0; n < S->N; ++n) if (S->owner[n] == j) { first = n; break; }
        js->node = first;
    }
    free(keep);
    js->gi = gi2; js->ci = ci2; js->g = g2; js->c = c2; js->m = m2;
    js->plan = plan; js->k = pl.cls >= 0 ? pl.np : k2; js->val = v; js->status = ST_RUNNING; js->cls = pl.cls;
    return 1;
}

/* CPU level an unallocated job starts its search at: its guaranteed minimum, else the lowest */
static int start_ci(const double *job) { return (int)job[JF_CMIN] > 0 ? (int)job[JF_CMIN] : 0; }

/* GPU / CPU increment the job would ask for next and its gain per unit of resource
 * (the slope of Section 5.2).  Target GPU level: the smallest level above the present one
 * whose curve value, at the job's CPU level and the top host-memory level, strictly
 * exceeds the job's present value.  Target CPU level: the next one.  Returns through
 * next[0..1] the level indices (-1 = none) and through gain[0..1] the gains. */
static void job_gains(const Sched *S, int j, const JobState *js, int32_t *next, double *gain)
{
    const double *job = S->jobs + (size_t)j * JF_COUNT;
    double w = job[JF_W];
    int mt = S->nM - 1;
    int allocated = js->gi >= 0;
    int ci = allocated ? js->ci : start_ci(job);
    double cur = allocated ? js->val : 0.0;
    next[0] = next[1] = -1; gain[0] = gain[1] = 0.0;
    for (int gi = js->gi + 1; gi < S->nG; ++gi) {
        double v = cval_of(S, js, cidx(S, j, gi, ci, mt));
        if (v > cur) {
            next[0] = gi;
            gain[0] = unit_gain(S, w, v, cur, (double)(S->g_levels[gi] - (allocated ? js->g : 0)));
            break;
        }
    }
    if (allocated && js->ci + 1 < S->nC) {
        double v = cval_of(S, js, cidx(S, j, js->gi, js->ci + 1, mt));
        double gn = unit_gain(S, w, v, cur, (double)(S->c_levels[js->ci + 1] - js->c));
        if (gn > 0.0) { next[1] = js->ci + 1; gain[1] = gn; }
    }
}

/* Marginal gains of every job for a given state (no placement test, no commit).
 * state_g / state_c / state_val: what each job holds (g = 0: nothing). */
void oracle_gain(const double *jobs, int J, const float *curve_val,
                 const int64_t *g_levels, int nG, const int64_t *c_levels, int nC, int nM,
                 const int64_t *state_g, const int64_t *state_c, const float *state_val,
                 float *gain_gpu, float *gain_cpu, int32_t *next_g, int32_t *next_c)
{
    Sched S; memset(&S, 0, sizeof S);
    S.J = J; S.nG = nG; S.nC = nC; S.nM = nM; S.cv = curve_val; S.jobs = jobs;
    S.g_levels = g_levels; S.c_levels = c_levels;
    for (int j = 0; j < J; ++j) {
        JobState js; memset(&js, 0, sizeof js);
        js.gi = -1; js.ci = 0; js.cls = -1;
        if (state_g[j] > 0) {
            for (int i = 0; i < nG; ++i) if (g_levels[i] == state_g[j]) js.gi = i;
            for (int i = 0; i < nC; ++i) if (c_levels[i] == state_c[j]) js.ci = i;
            js.g = state_g[j]; js.c = state_c[j]; js.val = state_val[j];
        }
        int32_t next[2]; double gain[2];
        job_gains(&S, j, &js, next, gain);
        gain_gpu[j] = (float)gain[0]; gain_cpu[j] = (float)gain[1]; next_g[j] = next[0]; next_c[j] = next[1];
    }
}

/* One scheduling round from an empty cluster of N identical nodes.
 * Phase A: jobs with a guaranteed minimum, in index order, are placed at it -- the paper's
 * "privileged" jobs: with tenant quotas (n_tenants > 0; quota[t] = GPUs, cores) only while the
 * minimum fits what is left of the job's tenant's quota, which a placed job then uses up
 * (Section 5.2: "the quota usage of each job [is] its minimum demand"); others stay pending.
 * Phase B: repeatedly take, among increments that can be placed, the largest positive
 * GPU gain (lowest job index on ties); when there is none, the largest positive CPU gain;
 * stop when there is neither or after max_steps increments were tried.
 * out_i: [J][8] = g, c, m_bytes, plan, first node, node count, status, m level of plan
 * out_val: [J] predicted throughput; node_out: [N][4] = free g, free c, free m, owner
 * step_log (optional, length max_steps): (job << 2) | (type << 1) | accepted.
 * Spread placement (optional, n_spread > 0; Section 5.2: a job's placement is a list of per-node allocations and
 * the plan is chosen for the placement found): when no single node takes a job of at most one node's GPUs, it is
 * assembled from free pieces of spread_align[k] GPUs on several nodes, in node order, for the first class k
 * that finds enough of them; the commit then reads class k's tables (predicted with the inter-node
 * bandwidth for every group that leaves a piece).  The gains of a job that sits in pieces are read off the
 * curves of its class; everybody else's off the packed curves.  out_pieces [J][32] / out_cls [J] report where such jobs sit.
 * curve_val64 (optional): the curve values in double precision; every decision is then taken in
 * double on that table and out_val64 (optional) receives the values unrounded.
 * cand_out (optional, [J][2][CAND_COUNT] doubles): what every job offered for the decision at which
 * the round stopped (the step the cap cut off, or the last look that found nothing): per resource
 * type the gain, the target level, whether it could be placed, the present and the target curve
 * value, the units added, whether the job was shut out (pending or frozen for that type), and what a
 * commit would read: the memory level that fits the target node(s) (-1: none), the curve value and
 * the GPU count of the curve entry there, and the (GPU level, core level) the increment leads to.
 * Returns the number of Phase-B steps, negated - 1 if the cap was hit first. */
enum { CAND_GAIN = 0, CAND_NEXT, CAND_PLACEABLE, CAND_VCUR, CAND_VNEXT, CAND_UNITS, CAND_SHUT, CAND_MCOMMIT, CAND_VCOMMIT, CAND_GCOMMIT, CAND_GI, CAND_CI, CAND_COUNT };

int oracle_round(const double *jobs, int J, const double *env,
                 const float *curve_val, const int32_t *curve_plan, const int32_t *curve_g,
                 const uint32_t *feas, int P,
                 const int64_t *g_levels, int nG, const int64_t *c_levels, int nC,
                 const int64_t *m_levels, int nM, int N, int max_steps,
                 const int64_t *quota, int n_tenants,
                 int64_t *out_i, float *out_val, int64_t *node_out, int32_t *step_log,
                 const double *curve_val64, double *out_val64, double *cand_out,
                 int n_spread, const int64_t *spread_align, const float *const *spread_val,
                 const int32_t *const *spread_plan, const int32_t *const *spread_g, const uint32_t *const *spread_feas,
                 int32_t *out_pieces, int32_t *out_cls)
{
    Sched S; memset(&S, 0, sizeof S);
    S.J = J; S.nG = nG; S.nC = nC; S.nM = nM; S.P = P; S.N = N;
    S.cv = curve_val; S.cv64 = curve_val64; S.cp = curve_plan; S.cg = curve_g; S.feas = feas; S.jobs = jobs;
    S.g_levels = g_levels; S.c_levels = c_levels; S.m_levels = m_levels;
    S.Gn = (int64_t)env[EF_GN]; S.Cn = (int64_t)env[EF_CN]; S.Mn = (int64_t)env[EF_MN];
    S.nK = n_spread; S.align = spread_align; S.kcv = spread_val; S.kcp = spread_plan; S.kcg = spread_g; S.kfeas = spread_feas;
    if (n_spread > 0) {
        S.piece_n = (int *)calloc((size_t)(J > 0 ? J : 1) * MAX_PIECES, sizeof(int));
        S.piece_q = (int *)calloc((size_t)(J > 0 ? J : 1) * MAX_PIECES, sizeof(int));
    }
    S.free_g = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    S.free_c = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    S.free_m = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    S.owner = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    for (int n = 0; n < N; ++n) { S.free_g[n] = S.Gn; S.free_c[n] = S.Cn; S.free_m[n] = S.Mn; S.owner[n] = -1; }
    JobState *st = (JobState *)calloc((size_t)(J > 0 ? J : 1), sizeof(JobState));
    for (int j = 0; j < J; ++j) { st[j].gi = -1; st[j].plan = -1; st[j].node = -1; st[j].status = ST_UNALLOCATED; st[j].cls = -1; }

    /* Phase A: guaranteed minima */
    int mt = nM - 1;
    int64_t *rem = NULL;
    if (n_tenants > 0) {
        rem = (int64_t *)malloc(sizeof(int64_t) * 2 * (size_t)n_tenants);
        memcpy(rem, quota, sizeof(int64_t) * 2 * (size_t)n_tenants);
    }
    for (int j = 0; j < J; ++j) {
        const double *job = jobs + (size_t)j * JF_COUNT;
        int gmin = (int)job[JF_GMIN];
        if (gmin < 0) continue;
        int cmin = start_ci(job);
        st[j].status = ST_PENDING;
        if (gmin >= nG || cmin >= nC) continue;
        size_t o = cidx(&S, j, gmin, cmin, mt);
        if (curve_plan[o] < 0) continue;
        /* the curve may reach this value with fewer GPUs than the level offers */
        int gi = -1;
        for (int i = 0; i < nG; ++i) if (g_levels[i] == (int64_t)curve_g[o]) gi = i;
        if (gi < 0) continue;
        int t = (int)job[JF_TENANT];
        if (n_tenants > 0) {
            if (t < 0 || t >= n_tenants) continue;
            if (rem[2 * t] < g_levels[gi] || rem[2 * t + 1] < c_levels[cmin]) continue;   /* beyond the quota: not privileged */
        }
        Place pl = find_place_of(&S, j, &st[j], g_levels[gi], c_levels[cmin]);
        if (!pl.ok) continue;
        commit(&S, j, &st[j], gi, cmin, pl, 0);
        if (st[j].gi < 0) st[j].status = ST_PENDING;
        else if (n_tenants > 0) { rem[2 * t] -= g_levels[gi]; rem[2 * t + 1] -= c_levels[cmin]; }
    }
    free(rem);

    /* Phase B: greedy increments */
    int steps = 0, capped = 0;
    for (;;) {
        int best_j = -1, best_type = -1, best_next = -1; double best_gain = 0.0;
        for (int type = 0; type < 2 && best_j < 0; ++type) {
            for (int j = 0; j < J; ++j) {
                if (st[j].status == ST_PENDING || st[j].frozen[type]) continue;
                int32_t next[2]; double gain[2];
                job_gains(&S, j, &st[j], next, gain);
                if (next[type] < 0 || !(gain[type] > 0.0)) continue;
                int gi2 = type == 0 ? next[0] : st[j].gi;
                int ci2 = type == 0 ? (st[j].gi >= 0 ? st[j].ci : start_ci(jobs + (size_t)j * JF_COUNT)) : next[1];
                Place pl = find_place_of(&S, j, &st[j], g_levels[gi2], c_levels[ci2]);
                if (!pl.ok) continue;
                if (gain[type] > best_gain) { best_gain = gain[type]; best_j = j; best_type = type; best_next = next[type]; }
            }
        }
        if (best_j < 0) break;
        if (steps >= max_steps) { capped = 1; break; }
        int j = best_j;
        int gi2 = best_type == 0 ? best_next : st[j].gi;
        int ci2 = best_type == 0 ? (st[j].gi >= 0 ? st[j].ci : start_ci(jobs + (size_t)j * JF_COUNT)) : best_next;
        Place pl = find_place_of(&S, j, &st[j], g_levels[gi2], c_levels[ci2]);
        int ok = commit(&S, j, &st[j], gi2, ci2, pl, 1);
        if (!ok) st[j].frozen[best_type] = 1;
        if (step_log) step_log[steps] = (int32_t)((j << 2) | (best_type << 1) | ok);
        ++steps;
    }

    /* what every job offered for the decision the round stopped at */
    if (cand_out)
        for (int j = 0; j < J; ++j) {
            int32_t next[2]; double gain[2];
            job_gains(&S, j, &st[j], next, gain);
            for (int type = 0; type < 2; ++type) {
                double *c = cand_out + ((size_t)j * 2 + type) * CAND_COUNT;
                for (int i = 0; i < CAND_COUNT; ++i) c[i] = 0.0;
                c[CAND_GAIN] = gain[type]; c[CAND_NEXT] = next[type];
                c[CAND_SHUT] = st[j].status == ST_PENDING || st[j].frozen[type];
                c[CAND_VCUR] = st[j].gi >= 0 ? st[j].val : 0.0;
                if (next[type] < 0) continue;
                int gi2 = type == 0 ? next[0] : st[j].gi;
                int ci2 = type == 0 ? (st[j].gi >= 0 ? st[j].ci : start_ci(jobs + (size_t)j * JF_COUNT)) : next[1];
                Place pl = find_place_of(&S, j, &st[j], g_levels[gi2], c_levels[ci2]);
                c[CAND_PLACEABLE] = pl.ok; c[CAND_GI] = gi2; c[CAND_CI] = ci2;
                c[CAND_MCOMMIT] = -1.0;
                if (pl.ok && (pl.k > 1 || pl.node >= 0)) {
                    int mi = commit_level(&S, &st[j], pl, g_levels[gi2]);
                    c[CAND_MCOMMIT] = mi;
                    if (mi >= 0 && pl.cls < 0) { c[CAND_VCOMMIT] = cval(&S, cidx(&S, j, gi2, ci2, mi)); c[CAND_GCOMMIT] = curve_g[cidx(&S, j, gi2, ci2, mi)]; }
                    if (mi >= 0 && pl.cls >= 0) { c[CAND_VCOMMIT] = spread_val[pl.cls][cidx(&S, j, gi2, ci2, mi)]; c[CAND_GCOMMIT] = spread_g[pl.cls][cidx(&S, j, gi2, ci2, mi)]; }
                }
                c[CAND_VNEXT] = cval(&S, cidx(&S, j, gi2, ci2, mt));
                c[CAND_UNITS] = type == 0 ? (double)(g_levels[gi2] - (st[j].gi >= 0 ? st[j].g : 0))
                                          : (double)(c_levels[ci2] - st[j].c);
            }
        }

    for (int j = 0; j < J; ++j) {
        int64_t *o = out_i + (size_t)j * 8;
        int alloc = st[j].gi >= 0;
        o[0] = alloc ? st[j].g : 0; o[1] = alloc ? st[j].c : 0; o[2] = alloc ? st[j].m : 0;
        o[3] = alloc ? st[j].plan : -1; o[4] = alloc ? st[j].node : -1; o[5] = alloc ? st[j].k : 0;
        o[6] = st[j].status;
        int f = -1;
        if (alloc) { uint32_t wd = feas[(size_t)j * P + st[j].plan]; f = 0; while (f < nM && !((wd >> f) & 1u)) ++f; }
        o[7] = f;
        out_val[j] = alloc ? (float)st[j].val : 0.0f;
        if (out_val64) out_val64[j] = alloc ? st[j].val : 0.0;
        /* where a spread job sits: node << 8 | GPUs there, ascending nodes; -1 = unused entry */
        if (out_cls) out_cls[j] = alloc ? st[j].cls : -1;
        if (out_pieces)
            for (int i = 0; i < MAX_PIECES; ++i)
                out_pieces[(size_t)j * MAX_PIECES + i] = (alloc && st[j].cls >= 0 && i < st[j].np)
                    ? (int32_t)((S.piece_n[(size_t)j * MAX_PIECES + i] << 8) | (int)(S.piece_q[(size_t)j * MAX_PIECES + i] * spread_align[st[j].cls])) : -1;
    }
    if (node_out)
        for (int n = 0; n < N; ++n) {
            node_out[(size_t)n * 4 + 0] = S.free_g[n]; node_out[(size_t)n * 4 + 1] = S.free_c[n];
            node_out[(size_t)n * 4 + 2] = S.free_m[n]; node_out[(size_t)n * 4 + 3] = S.owner[n];
        }
    free(S.free_g); free(S.free_c); free(S.free_m); free(S.owner); free(st); free(S.piece_n); free(S.piece_q);
    return capped ? -steps - 1 : steps;
}

/* ======================================================================================
 * Incremental round: Algorithm 1 with its shrink step, started from the previous allocation
 * (Section 5.2 "Scheduling algorithm design" and "Incorporating reconfiguration penalty").
 *
 * Reading (the paper leaves the step size, the order of attempts and the roll-back open):
 *  - Job slots keep their index between rounds; active[j] = 0 marks an empty slot.  A job
 *    whose previous status is RUNNING keeps its GPUs, cores, memory, plan and node(s).
 *  - Gate: a running job may be touched only if T > 0 and (T - (N + 1) * delta) / T > theta
 *    (T seconds trained, N reconfigurations so far, delta seconds per checkpoint-resume; the
 *    contemplated reconfiguration is counted).  Otherwise it is pinned: it neither grows nor
 *    shrinks in this round.
 *  - Minimum of a guaranteed job: the GPU count the curve really uses at (gmin, cmin), and cmin
 *    cores.  Best-effort jobs have none.
 *  - Shrink step of a running, unpinned single-node job ("over its minimum"): GPUs go down to the
 *    next lower level whose own plans run (not below the minimum; a best-effort job without such
 *    a level is preempted: everything released, back to the queue); cores go down one level (not
 *    below the minimum, never to zero).  Its slope is the weighted value lost per unit given up,
 *    read at the top memory level like the gains.  The shrunk job's plan and memory are
 *    re-selected on its node (GetBestPlan / AllocMem); a step that does not fit is not offered.
 *  - Exchange for an increment of job j on node n: while the node lacks GPUs (then cores) for
 *    it, shrink the offered job on n with the lowest slope (lowest index on ties), provided the
 *    slope is below j's gain for that resource, or unconditionally while j is a guaranteed job
 *    being placed at its minimum.  A running job may reclaim only the resource of its
 *    increment; a queued job pre-allocates GPUs and cores together, so its value per GPU and
 *    per core are its two gains.  At most MAX_EXCHANGE shrink steps; then j is committed on n.  Any failure undoes the whole attempt.  Shrunk jobs do not grow again in the round.
 *  - Phase A: queued guaranteed jobs in index order, within what their tenant's quota leaves
 *    after the minima of its running guaranteed jobs, are placed at their minimum: free
 *    resources first (first fit), else by exchange on the first node where it succeeds.
 *  - Phase B: as in the grow-only round while some increment fits free resources.  When none
 *    does, the largest-gain increment that is not frozen (GPU before CPU, lowest index on ties)
 *    tries an exchange: a running single-node job on its own node, a queued job on the first node
 *    where it succeeds; increments above one node never exchange.  Failure freezes (job, type).
 *  step_log entry: (job << 3) | (by exchange << 2) | (type << 1) | accepted.
 * ==================================================================================== */
#define MAX_EXCHANGE 64

typedef struct { int ok; int gi2, ci2; float slope; } Shrink;

/* what job v would give up next of resource `type`, and at what loss per unit */
static Shrink shrink_option(const Sched *S, int v, const JobState *js, int type, int guaranteed, int min_gi, int min_ci)
{
    Shrink sh; sh.ok = 0; sh.gi2 = -1; sh.ci2 = js->ci; sh.slope = 0.0f;
    if (js->gi < 0 || js->k != 1) return sh;
    const double *job = S->jobs + (size_t)v * JF_COUNT;
    float w = (float)job[JF_W];
    int mt = S->nM - 1;
    float vcur = w * (float)js->val;
    if (type == 0) {
        if (guaranteed && min_gi < 0) return sh;
        int lo = guaranteed ? min_gi : 0;
        for (int i = js->gi - 1; i >= lo; --i) {
            size_t o = cidx(S, v, i, js->ci, mt);
            if (S->cp[o] >= 0 && (int64_t)S->cg[o] == S->g_levels[i]) {
                sh.ok = 1; sh.gi2 = i;
                sh.slope = (vcur - w * S->cv[o]) / (float)(js->g - S->g_levels[i]);
                return sh;
            }
        }
        if (guaranteed) return sh;
        sh.ok = 1; sh.gi2 = -1;                      /* preemption */
        sh.slope = (vcur - w * 0.0f) / (float)js->g;
        return sh;
    }
    int lo = guaranteed ? min_ci : 0;
    if (js->ci - 1 < lo) return sh;
    size_t o = cidx(S, v, js->gi, js->ci - 1, mt);
    if (S->cp[o] < 0 || (int64_t)S->cg[o] != js->g) return sh;
    sh.ok = 1; sh.gi2 = js->gi; sh.ci2 = js->ci - 1;
    sh.slope = (vcur - w * S->cv[o]) / (float)(js->c - S->c_levels[js->ci - 1]);
    return sh;
}

/* performs the shrink step (apply != 0) or only tells whether it fits (apply == 0) */
static int do_shrink(Sched *S, int v, JobState *js, Shrink sh, int apply)
{
    if (sh.gi2 < 0) {
        if (apply) {
            release_job(S, v, js);
            js->gi = -1; js->ci = 0; js->g = js->c = js->m = 0; js->plan = -1; js->node = -1; js->k = 0; js->cls = -1;
            js->val = 0.0; js->status = ST_UNALLOCATED;
        }
        return 1;
    }
    int n = js->node;
    int64_t fg = S->free_g[n], fc = S->free_c[n], fm = S->free_m[n];
    JobState keep = *js;
    Place pl; pl.ok = 1; pl.k = 1; pl.stay = 1; pl.node = n; pl.need_new = 0; pl.cls = -1; pl.np = 0;
    int ok = commit(S, v, js, sh.gi2, sh.ci2, pl, 0);
    if (!ok || !apply) { S->free_g[n] = fg; S->free_c[n] = fc; S->free_m[n] = fm; *js = keep; }
    return ok;
}

typedef struct { const int *pinned, *guaranteed, *min_gi, *min_ci; } Roles;

static int exchange(Sched *S, JobState *st, const Roles *R, int j, int gi2, int ci2, int n,
                    int force, const float *cand_gain, int need_gain)
{
    int J = S->J, N = S->N;
    JobState *st0 = (JobState *)malloc(sizeof(JobState) * (size_t)J);
    int64_t *node0 = (int64_t *)malloc(sizeof(int64_t) * 3 * (size_t)N);
    int32_t *own0 = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    memcpy(st0, st, sizeof(JobState) * (size_t)J);
    memcpy(node0, S->free_g, sizeof(int64_t) * (size_t)N);
    memcpy(node0 + N, S->free_c, sizeof(int64_t) * (size_t)N);
    memcpy(node0 + 2 * N, S->free_m, sizeof(int64_t) * (size_t)N);
    memcpy(own0, S->owner, sizeof(int32_t) * (size_t)N);

    int on_n = st[j].gi >= 0 && st[j].k == 1 && st[j].node == n;
    int64_t need[2];
    need[0] = S->g_levels[gi2] - (on_n ? st[j].g : 0);
    need[1] = S->c_levels[ci2] - (on_n ? st[j].c : 0);
    int ok = 1, taken = 0;
    for (int r = 0; r < 2 && ok; ++r) {
        int64_t *free_r = r == 0 ? S->free_g : S->free_c;
        while (free_r[n] < need[r]) {
            if (!force && !(cand_gain[r] > 0.0f)) { ok = 0; break; }    /* this resource may not be reclaimed */
            int best = -1; Shrink best_sh; best_sh.slope = 0.0f;
            for (int v = 0; v < J; ++v) {
                if (v == j || st[v].gi < 0 || st[v].k != 1 || st[v].node != n || R->pinned[v]) continue;
                Shrink sh = shrink_option(S, v, &st[v], r, R->guaranteed[v], R->min_gi[v], R->min_ci[v]);
                if (!sh.ok || !do_shrink(S, v, &st[v], sh, 0)) continue;
                if (best < 0 || sh.slope < best_sh.slope) { best = v; best_sh = sh; }
            }
            if (best < 0) { ok = 0; break; }
            if (!force && !(cand_gain[r] > best_sh.slope)) { ok = 0; break; }
            if (++taken > MAX_EXCHANGE) { ok = 0; break; }
            do_shrink(S, best, &st[best], best_sh, 1);
            st[best].frozen[0] = st[best].frozen[1] = 1;
        }
    }
    if (ok) {
        Place pl; pl.ok = 1; pl.k = 1; pl.stay = on_n; pl.node = n; pl.need_new = 0; pl.cls = -1; pl.np = 0;
        ok = commit(S, j, &st[j], gi2, ci2, pl, need_gain);
    }
    if (!ok) {
        memcpy(st, st0, sizeof(JobState) * (size_t)J);
        memcpy(S->free_g, node0, sizeof(int64_t) * (size_t)N);
        memcpy(S->free_c, node0 + N, sizeof(int64_t) * (size_t)N);
        memcpy(S->free_m, node0 + 2 * N, sizeof(int64_t) * (size_t)N);
        memcpy(S->owner, own0, sizeof(int32_t) * (size_t)N);
    }
    free(st0); free(node0); free(own0);
    return ok;
}

/* prev_i [J][8], prev_val [J]: the previous round's out_i / out_val (status RUNNING = carried
 * over); prev_owner [N]: its node owners; active [J]; T, delta [J] seconds; nrec [J]
 * reconfigurations so far; theta: the gate's threshold (the paper uses 0.97).
 * Outputs as oracle_round.  Returns the number of Phase-B steps, negated - 1 if capped;
 * INT32_MIN when the previous state does not fit the grid or the cluster. */
int oracle_round_incremental(const double *jobs, int J, const double *env,
                             const float *curve_val, const int32_t *curve_plan, const int32_t *curve_g,
                             const uint32_t *feas, int P,
                             const int64_t *g_levels, int nG, const int64_t *c_levels, int nC,
                             const int64_t *m_levels, int nM, int N, int max_steps,
                             const int64_t *quota, int n_tenants,
                             const int64_t *prev_i, const float *prev_val, const int32_t *prev_owner,
                             const int32_t *active, const float *T, const float *delta, const int32_t *nrec,
                             float theta,
                             int64_t *out_i, float *out_val, int64_t *node_out, int32_t *step_log)
{
    Sched S; memset(&S, 0, sizeof S);
    S.J = J; S.nG = nG; S.nC = nC; S.nM = nM; S.P = P; S.N = N;
    S.cv = curve_val; S.cp = curve_plan; S.cg = curve_g; S.feas = feas; S.jobs = jobs;
    S.g_levels = g_levels; S.c_levels = c_levels; S.m_levels = m_levels;
    S.Gn = (int64_t)env[EF_GN]; S.Cn = (int64_t)env[EF_CN]; S.Mn = (int64_t)env[EF_MN];
    S.free_g = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    S.free_c = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    S.free_m = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    S.owner = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    for (int n = 0; n < N; ++n) { S.free_g[n] = S.Gn; S.free_c[n] = S.Cn; S.free_m[n] = S.Mn; S.owner[n] = -1; }
    size_t Jn = (size_t)(J > 0 ? J : 1);
    JobState *st = (JobState *)calloc(Jn, sizeof(JobState));
    int *pinned = (int *)calloc(Jn, sizeof(int)), *guaranteed = (int *)calloc(Jn, sizeof(int));
    int *min_gi = (int *)calloc(Jn, sizeof(int)), *min_ci = (int *)calloc(Jn, sizeof(int));
    Roles R; R.pinned = pinned; R.guaranteed = guaranteed; R.min_gi = min_gi; R.min_ci = min_ci;
    int mt = nM - 1, bad = 0;

    /* carried state, minima, gate */
    for (int j = 0; j < J; ++j) {
        const double *job = jobs + (size_t)j * JF_COUNT;
        st[j].gi = -1; st[j].plan = -1; st[j].node = -1; st[j].status = ST_UNALLOCATED; st[j].cls = -1;
        guaranteed[j] = (int)job[JF_GMIN] >= 0;
        min_gi[j] = -1; min_ci[j] = start_ci(job);
        if (guaranteed[j] && (int)job[JF_GMIN] < nG && min_ci[j] < nC) {
            size_t o = cidx(&S, j, (int)job[JF_GMIN], min_ci[j], mt);
            if (curve_plan[o] >= 0)
                for (int i = 0; i < nG; ++i) if (g_levels[i] == (int64_t)curve_g[o]) min_gi[j] = i;
        }
        if (!active[j] || prev_i[(size_t)j * 8 + 6] != ST_RUNNING) continue;
        const int64_t *pv = prev_i + (size_t)j * 8;
        int gi = -1, ci = -1;
        for (int i = 0; i < nG; ++i) if (g_levels[i] == pv[0]) gi = i;
        for (int i = 0; i < nC; ++i) if (c_levels[i] == pv[1]) ci = i;
        int k = (int)pv[5];
        if (gi < 0 || ci < 0 || pv[3] < 0 || pv[3] >= P || pv[4] < 0 || pv[4] >= N || k < 1
            || (k == 1 ? pv[0] > S.Gn : pv[0] != (int64_t)k * S.Gn)
            || pv[7] < 0 || pv[7] >= nM || m_levels[pv[7]] != pv[2]) { bad = 1; continue; }
        st[j].gi = gi; st[j].ci = ci; st[j].g = pv[0]; st[j].c = pv[1]; st[j].m = pv[2];
        st[j].plan = (int)pv[3]; st[j].node = (int)pv[4]; st[j].k = k; st[j].val = prev_val[j];
        st[j].status = ST_RUNNING;
        if (k == 1) {
            int n = st[j].node;
            S.free_g[n] -= st[j].g; S.free_c[n] -= st[j].c; S.free_m[n] -= st[j].m;
        } else {
            int cnt = 0;
            for (int n = 0; n < N; ++n)
                if (prev_owner[n] == j) {
                    S.free_g[n] -= S.Gn; S.free_c[n] -= cdiv(st[j].c, k); S.free_m[n] -= cdiv(st[j].m, k);
                    S.owner[n] = j; ++cnt;
                }
            if (cnt != k) bad = 1;
        }
        float t = T[j];
        int pass = t > 0.0f && (t - (float)(nrec[j] + 1) * delta[j]) / t > theta;
        pinned[j] = !pass;
    }
    for (int n = 0; n < N; ++n) if (S.free_g[n] < 0 || S.free_c[n] < 0 || S.free_m[n] < 0) bad = 1;
    if (bad) {
        free(S.free_g); free(S.free_c); free(S.free_m); free(S.owner); free(st);
        free(pinned); free(guaranteed); free(min_gi); free(min_ci);
        return INT32_MIN;
    }

    /* Phase A: queued guaranteed jobs within their tenant's remaining quota */
    int64_t *rem = NULL;
    if (n_tenants > 0) {
        rem = (int64_t *)malloc(sizeof(int64_t) * 2 * (size_t)n_tenants);
        memcpy(rem, quota, sizeof(int64_t) * 2 * (size_t)n_tenants);
        for (int j = 0; j < J; ++j) {
            int t = (int)jobs[(size_t)j * JF_COUNT + JF_TENANT];
            if (st[j].gi >= 0 && guaranteed[j] && min_gi[j] >= 0 && t >= 0 && t < n_tenants) {
                rem[2 * t] -= g_levels[min_gi[j]]; rem[2 * t + 1] -= c_levels[min_ci[j]];
            }
        }
    }
    for (int j = 0; j < J; ++j) {
        if (!active[j] || !guaranteed[j] || st[j].gi >= 0) continue;
        st[j].status = ST_PENDING;
        if (min_gi[j] < 0) continue;
        int gi = min_gi[j], cmin = min_ci[j];
        int t = (int)jobs[(size_t)j * JF_COUNT + JF_TENANT];
        if (n_tenants > 0) {
            if (t < 0 || t >= n_tenants) continue;
            if (rem[2 * t] < g_levels[gi] || rem[2 * t + 1] < c_levels[cmin]) continue;
        }
        Place pl = find_place_of(&S, j, &st[j], g_levels[gi], c_levels[cmin]);
        int placed = pl.ok && commit(&S, j, &st[j], gi, cmin, pl, 0);
        if (!placed && g_levels[gi] <= S.Gn)
            for (int n = 0; n < N && !placed; ++n)
                placed = exchange(&S, st, &R, j, gi, cmin, n, 1, NULL, 0);
        if (!placed) { st[j].status = ST_PENDING; continue; }
        if (n_tenants > 0) { rem[2 * t] -= g_levels[gi]; rem[2 * t + 1] -= c_levels[cmin]; }
    }
    free(rem);

    /* Phase B */
    int steps = 0, capped = 0;
    for (;;) {
        int best_j = -1, best_type = -1, best_next = -1, by_exchange = 0; double best_gain = 0.0;
        for (int pass = 0; pass < 2 && best_j < 0; ++pass)          /* 0: fits free resources; 1: any */
            for (int type = 0; type < 2 && best_j < 0; ++type)
                for (int j = 0; j < J; ++j) {
                    if (!active[j] || pinned[j] || st[j].status == ST_PENDING || st[j].frozen[type]) continue;
                    int32_t next[2]; double gain[2];
                    job_gains(&S, j, &st[j], next, gain);
                    if (next[type] < 0 || !(gain[type] > 0.0)) continue;
                    if (pass == 0) {
                        int gi2 = type == 0 ? next[0] : st[j].gi;
                        int ci2 = type == 0 ? (st[j].gi >= 0 ? st[j].ci : start_ci(jobs + (size_t)j * JF_COUNT)) : next[1];
                        Place pl = find_place_of(&S, j, &st[j], g_levels[gi2], c_levels[ci2]);
                        if (!pl.ok) continue;
                    }
                    if (gain[type] > best_gain) { best_gain = gain[type]; best_j = j; best_type = type; best_next = next[type]; by_exchange = pass; }
                }
        if (best_j < 0) break;
        if (steps >= max_steps) { capped = 1; break; }
        int j = best_j;
        int gi2 = best_type == 0 ? best_next : st[j].gi;
        int ci2 = best_type == 0 ? (st[j].gi >= 0 ? st[j].ci : start_ci(jobs + (size_t)j * JF_COUNT)) : best_next;
        int ok = 0;
        if (!by_exchange) {
            Place pl = find_place_of(&S, j, &st[j], g_levels[gi2], c_levels[ci2]);
            ok = commit(&S, j, &st[j], gi2, ci2, pl, 1);
        } else if (g_levels[gi2] <= S.Gn) {
            /* what j gains per unit of each resource it would take from others: a running job only
             * asks for the resource of its increment; a queued job pre-allocates GPUs and cores
             * together, so its value counts per GPU and per core */
            float cand[2] = {0.0f, 0.0f};
            cand[best_type] = (float)best_gain;
            if (st[j].gi >= 0) {
                if (st[j].k == 1) ok = exchange(&S, st, &R, j, gi2, ci2, st[j].node, 0, cand, 1);
            } else {
                float w = (float)jobs[(size_t)j * JF_COUNT + JF_W];
                cand[1] = (w * curve_val[cidx(&S, j, gi2, ci2, mt)] - 0.0f) / (float)c_levels[ci2];
                for (int n = 0; n < N && !ok; ++n)
                    ok = exchange(&S, st, &R, j, gi2, ci2, n, 0, cand, 1);
            }
        }
        if (!ok) st[j].frozen[best_type] = 1;
        if (step_log) step_log[steps] = (int32_t)((j << 3) | (by_exchange << 2) | (best_type << 1) | ok);
        ++steps;
    }

    for (int j = 0; j < J; ++j) {
        int64_t *o = out_i + (size_t)j * 8;
        int alloc = st[j].gi >= 0;
        o[0] = alloc ? st[j].g : 0; o[1] = alloc ? st[j].c : 0; o[2] = alloc ? st[j].m : 0;
        o[3] = alloc ? st[j].plan : -1; o[4] = alloc ? st[j].node : -1; o[5] = alloc ? st[j].k : 0;
        o[6] = st[j].status;
        int f = -1;
        if (alloc) { uint32_t wd = feas[(size_t)j * P + st[j].plan]; f = 0; while (f < nM && !((wd >> f) & 1u)) ++f; }
        o[7] = f;
        out_val[j] = alloc ? (float)st[j].val : 0.0f;
    }
    if (node_out)
        for (int n = 0; n < N; ++n) {
            node_out[(size_t)n * 4 + 0] = S.free_g[n]; node_out[(size_t)n * 4 + 1] = S.free_c[n];
            node_out[(size_t)n * 4 + 2] = S.free_m[n]; node_out[(size_t)n * 4 + 3] = S.owner[n];
        }
    free(S.free_g); free(S.free_c); free(S.free_m); free(S.owner); free(st);
    free(pinned); free(guaranteed); free(min_gi); free(min_ci);
    return capped ? -steps - 1 : steps;
}

/* ======================================================================================
 * Section 4.3, "Continuous model fitting": the seven fittable parameters of a model type
 * (k_bwd, k_sync, k_opt, k_opt_off, k_off, k_swap, k_const) are chosen to minimise the root
 * mean squared logarithmic error between the model and throughputs measured on sampled
 * (plan, cores) configurations:  RMSLE = sqrt(mean_i (ln(1 + pred_i) - ln(1 + y_i))^2).
 *
 * The paper names no optimiser.  This project's reading is a derivative-free pattern search
 * that two implementations can follow decision by decision:
 *  - start from the coefficients in the job record (the previous fit), clamped to the bounds;
 *  - `sweeps` sweeps; sweep r moves one parameter at a time, in Table 1's order, among the values
 *    base * M_r^e, e = -4 .. 4, clamped, where M_0 = 2^(3/4) and M_(r+1) = sqrt(M_r); the other
 *    six stay at their latest values; the candidate with the smallest error wins, the present
 *    value on ties, then candidates in the order e = -1, +1, -2, +2, ... ;
 *  - candidate values are built from correctly rounded operations only (sqrt, *, /), so they are
 *    the same numbers everywhere; only the model's own pow / log may differ in the last bits.
 * out_theta [J][7]; out_rmsle [J][2] = before, after; out_margin [J] = the smallest relative gap
 * between the winning and the next distinct error over all decisions of the fit (a second
 * implementation may only deviate where this is tiny).
 * ==================================================================================== */
enum { FIT_PARAMS = 7 };
static const int fit_field[FIT_PARAMS] = {JF_KBWD, JF_KSYNC, JF_KOPT, JF_KOPTOFF, JF_KOFF, JF_KSWAP, JF_KCONST};
static const double fit_lo[FIT_PARAMS] = {0.25, 1.0, 1e-13, 1e-10, 1.0, 1.0, 1e-4};
static const double fit_hi[FIT_PARAMS] = {16.0, 16.0, 1e-9, 1e-6, 16.0, 16.0, 10.0};

static double fit_sse(const double *row, const double *env, const int32_t *plans,
                      const int32_t *s_plan, const int64_t *s_c, const double *s_thr, int S, int *n_out)
{
    double sse = 0.0; int n = 0;
    for (int i = 0; i < S; ++i) {
        if (s_plan[i] < 0) continue;
        double out[TF_COUNT];
        oracle_terms(row, env, plans + (size_t)s_plan[i] * PF_COUNT, (double)s_c[i], out);
        double e = log1p(out[TF_THR]) - log1p(s_thr[i]);
        sse += e * e; ++n;
    }
    if (n_out) *n_out = n;
    return sse;
}

#define FIT_EPS 1e-9      /* a move must lower the squared error by more than this fraction */

void oracle_fit(const double *jobs, int J, const double *env, const int32_t *plans, int P,
                const int32_t *s_plan, const int64_t *s_c, const double *s_thr, int S, int sweeps,
                double *out_theta, double *out_rmsle, double *out_margin)
{
    (void)P;
    static const int order[8] = {-1, 1, -2, 2, -3, 3, -4, 4};
    for (int j = 0; j < J; ++j) {
        double row[JF_COUNT];
        memcpy(row, jobs + (size_t)j * JF_COUNT, sizeof row);
        const int32_t *sp = s_plan + (size_t)j * S; const int64_t *sc = s_c + (size_t)j * S; const double *sy = s_thr + (size_t)j * S;
        for (int p = 0; p < FIT_PARAMS; ++p) {
            double v = row[fit_field[p]];
            if (!(v >= fit_lo[p])) v = fit_lo[p];
            if (v > fit_hi[p]) v = fit_hi[p];
            row[fit_field[p]] = v;
        }
        int n = 0;
        double cur = fit_sse(row, env, plans, sp, sc, sy, S, &n);
        double margin = INFINITY;
        out_rmsle[2 * j] = n > 0 ? sqrt(cur / n) : 0.0;
        double M = sqrt(2.0) * sqrt(sqrt(2.0));                 /* 2^(3/4) */
        for (int r = 0; r < sweeps && n > 0; ++r) {
            double mul[5]; mul[0] = 1.0; mul[1] = M; mul[2] = M * M; mul[3] = mul[2] * M; mul[4] = mul[2] * mul[2];
            double before[FIT_PARAMS];
            for (int p = 0; p < FIT_PARAMS; ++p) before[p] = row[fit_field[p]];
            /* exploratory moves, one parameter at a time */
            for (int p = 0; p < FIT_PARAMS; ++p) {
                double base = row[fit_field[p]];
                double best = cur, best_v = base;
                for (int q = 0; q < 8; ++q) {
                    int e = order[q];
                    double v = e > 0 ? base * mul[e] : base / mul[-e];
                    if (v < fit_lo[p]) v = fit_lo[p];
                    if (v > fit_hi[p]) v = fit_hi[p];
                    if (v == base) continue;
                    row[fit_field[p]] = v;
                    double sse = fit_sse(row, env, plans, sp, sc, sy, S, NULL);
                    double bar = best * (1.0 - FIT_EPS);
                    double gap = fabs(sse - bar) / (bar > 1e-300 ? bar : 1e-300);
                    if (gap < margin) margin = gap;
                    if (sse < bar) { best = sse; best_v = v; }
                }
                row[fit_field[p]] = best_v; cur = best;
            }
            /* pattern moves (Hooke and Jeeves): repeat the sweep's combined displacement while it pays */
            for (int rep = 0; rep < 4; ++rep) {
                double keep[FIT_PARAMS]; int moved = 0;
                for (int p = 0; p < FIT_PARAMS; ++p) {
                    keep[p] = row[fit_field[p]];
                    double v = keep[p] * keep[p] / before[p];
                    if (v < fit_lo[p]) v = fit_lo[p];
                    if (v > fit_hi[p]) v = fit_hi[p];
                    if (v != keep[p]) moved = 1;
                    row[fit_field[p]] = v;
                }
                if (!moved) break;
                double sse = fit_sse(row, env, plans, sp, sc, sy, S, NULL);
                double bar = cur * (1.0 - FIT_EPS);
                double gap = fabs(sse - bar) / (bar > 1e-300 ? bar : 1e-300);
                if (gap < margin) margin = gap;
                if (sse < bar) { cur = sse; for (int p = 0; p < FIT_PARAMS; ++p) before[p] = keep[p]; }
                else { for (int p = 0; p < FIT_PARAMS; ++p) row[fit_field[p]] = keep[p]; break; }
            }
            if (r & 1) M = sqrt(M);                             /* the step halves every second sweep */
        }
        for (int p = 0; p < FIT_PARAMS; ++p) out_theta[(size_t)j * FIT_PARAMS + p] = row[fit_field[p]];
        out_rmsle[2 * j + 1] = n > 0 ? sqrt(cur / n) : 0.0;
        out_margin[j] = margin;
    }
}

/* Exhaustive search on one node (tiny instances only): every job is either left out or
 * given one (g level, c level, m level); the allocation uses the GPUs of the curve entry,
 * the cores of the level and the memory of the entry's plan; sums must fit the node.
 * Returns the largest total weighted throughput (double accumulation of w * value, the
 * products taken in single precision as in the greedy round). */
typedef struct { float v; int64_t g, c, m; } Opt;

static void bf_rec(int j, int J, const Opt *opts, const int *nopt, int maxopt,
                   int64_t rg, int64_t rc, int64_t rm, double acc, double *best)
{
    if (j == J) { if (acc > *best) *best = acc; return; }
    bf_rec(j + 1, J, opts, nopt, maxopt, rg, rc, rm, acc, best);
    for (int i = 0; i < nopt[j]; ++i) {
        const Opt *o = &opts[(size_t)j * maxopt + i];
        if (o->g <= rg && o->c <= rc && o->m <= rm)
            bf_rec(j + 1, J, opts, nopt, maxopt, rg - o->g, rc - o->c, rm - o->m, acc + (double)o->v, best);
    }
}

double oracle_bruteforce(const double *jobs, int J, const double *env,
                         const float *curve_val, const int32_t *curve_plan, const int32_t *curve_g,
                         const uint32_t *feas, int P,
                         const int64_t *g_levels, int nG, const int64_t *c_levels, int nC,
                         const int64_t *m_levels, int nM)
{
    int maxopt = nG * nC * nM;
    Opt *opts = (Opt *)malloc(sizeof(Opt) * (size_t)maxopt * (size_t)(J > 0 ? J : 1));
    int *nopt = (int *)calloc((size_t)(J > 0 ? J : 1), sizeof(int));
    (void)g_levels;
    for (int j = 0; j < J; ++j) {
        float w = (float)jobs[(size_t)j * JF_COUNT + JF_W];
        for (int gi = 0; gi < nG; ++gi)
            for (int ci = 0; ci < nC; ++ci)
                for (int mi = 0; mi < nM; ++mi) {
                    size_t o = (((size_t)j * nG + gi) * nC + ci) * nM + mi;
                    if (curve_plan[o] < 0) continue;
                    uint32_t wd = feas[(size_t)j * P + curve_plan[o]];
                    int f = 0; while (f < nM && !((wd >> f) & 1u)) ++f;
                    if (f > mi) continue;
                    Opt *op = &opts[(size_t)j * maxopt + nopt[j]++];
                    op->v = w * curve_val[o]; op->g = curve_g[o]; op->c = c_levels[ci]; op->m = m_levels[f];
                }
    }
    double best = 0.0;
    bf_rec(0, J, opts, nopt, maxopt, (int64_t)env[EF_GN], (int64_t)env[EF_CN], (int64_t)env[EF_MN], 0.0, &best);
    free(opts); free(nopt);
    return best;
}
