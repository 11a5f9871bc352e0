// Internal declarations shared by the translation units of librubick (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <string>
#include <vector>

#include "rubick.h"

namespace rubick {

// Per plan quad (four consecutive plans sharing d, t, p and the ZeRO stage), packed for the
// evaluation kernel.  Built by rubick_set_space from the plan list and the environment.
struct QuadDesc {
    uint8_t log2d, log2t, log2p, zero;
    uint8_t g_level;
    uint8_t flags;      // QF_* bits
    uint8_t disabled;   // bit i: plan 4q + i is disabled
    uint8_t pad;
};
enum : uint8_t {
    QF_T_FITS_NODE = 1,   // t <= gpus_per_node
    QF_DP_INTER = 2,      // the data-parallel ring crosses nodes (d * t > gpus_per_node)
    QF_PP_INTER = 4,      // the pipeline crosses nodes (g > gpus_per_node)
};

// A plan quad of the wide plan space (degrees of any size), 16 bytes, read as one uint4:
// x = d | t << 16, y = p | ZeRO stage << 16 | micro-batch halvings << 24, z = QF_* flags | disabled bits << 8, w = 0.
struct WideQuad { uint32_t x, y, z, w; };

// Everything a kernel needs to know about the environment and the grid; passed by value as a
// __grid_constant__ kernel parameter so that level lookups are uniform constant-bank reads.
struct Space {
    int32_t P, Q;                 // plans, quads (P / 4)
    int32_t nG, nC, nM;
    int32_t Gn, log2Gn, Cn;
    int32_t strict;
    float z3_volume;              // factor on V_dp for ZeRO stage 3: 1 (Section 4.1's rule) or 1.5 (option)
    int32_t wide;                 // plans with degrees of any size (wide quad table) instead of powers of two
    int32_t n_small;              // number of GPU levels <= Gn (they come first)
    float e;                      // bytes per element
    float inv_B_intra, inv_B_inter, inv_B_pcie;
    int64_t gpu_mem, Mn;
    int32_t g_levels[RUBICK_MAX_G_LEVELS];
    int32_t group_off[RUBICK_MAX_G_LEVELS + 1];
    int32_t c_levels[RUBICK_MAX_C_LEVELS];
    float inv_c[RUBICK_MAX_C_LEVELS];
    int64_t m_levels[RUBICK_MAX_M_LEVELS];
};

// device status word bits (read back by rubick_sync / the round)
enum : uint32_t {
    DS_FEAS_NOT_THRESHOLD = 1u,
    DS_STEP_CAP = 2u,
    DS_BAD_PREV = 4u,             // incremental round: the previous state does not fit the grid or the cluster
};

// kernels launched by this process so far (every launch site counts itself; read by rubick_kernel_launches)
extern std::atomic<unsigned long long> g_kernel_launches;
inline void count_launch(int n = 1) { g_kernel_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

bool round_fast_supported(const Space &sp, int J, int N);
size_t round_fast_scratch_need(const Space &sp, int J, int N);
cudaError_t launch_round_fast(const Space &sp, const rubick_job *d_jobs, int J, const float *d_cv, const int32_t *d_cp,
                              const int32_t *d_cg, const uint32_t *d_feas, int N, int max_steps,
                              rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                              void *d_scratch, const int32_t *d_quota, int n_tenants,
                              uint32_t *d_status, int32_t *d_steps, cudaStream_t st, const int4 *d_top = nullptr);

}  // namespace rubick

// one plan with its degrees written out (both plan record formats are brought to this form)
struct NormPlan { int d, t, p, zero, gc, off, g_level, disabled, accum; };

struct rubick_ctx {
    rubick_env env;
    int device;
    cudaStream_t stream;
    bool has_space;
    rubick::Space space;
    std::vector<rubick_plan> plans;
    std::vector<NormPlan> norm_plans;   // the installed plan list (rubick_set_placement rebuilds the quad tables from it)
    int placement_align;                // placement class of the quad tables on the device: 0 packed, a > 0 spread
    rubick::QuadDesc *d_quads;          // [Q]
    rubick::WideQuad *d_wide_quads;     // [Q] only for a wide plan space
    uint32_t *d_status;                 // one word, DS_* bits
    int32_t *d_steps;                   // one word, steps of the last round
    int32_t *d_quota;                   // [2 * RUBICK_MAX_TENANTS] per tenant: GPUs, cores (uploaded per round)
    std::vector<int32_t> h_quota;       // staging copy that outlives the asynchronous upload
    // scratch of the greedy round (hot per-job state when it does not fit shared memory)
    void *d_round_scratch;
    size_t round_scratch_bytes;
    // scratch tables of rubick_schedule_round
    float *d_thr; uint32_t *d_feas; float *d_cv; int32_t *d_cp; int32_t *d_cg;
    size_t cap_thr, cap_feas, cap_curve;     // capacities in elements
    int4 *d_top; size_t cap_top;             // top-memory-level entries of the curves in context scratch, packed
    rubick_job *d_jobs_stage; size_t cap_jobs;
    rubick_assignment *d_out_stage; size_t cap_out;
    rubick_node *d_node_stage; size_t cap_node;
    int32_t *d_best_todo; size_t cap_best_todo;     // rubick_best_plan: count + jobs left to the general kernel
    // state that rubick_incremental_event_host carries from one event to the next
    int inc_J, inc_N;                   // slots / nodes of the carried state and of the cached tables; inc_J = 0: none
    int inc_cur;                        // which of the two state buffers holds the last result
    rubick_assignment *d_inc_state[2]; rubick_node *d_inc_nodes[2]; rubick_reconf *d_inc_reconf; rubick_job *d_inc_jobs;
    size_t cap_inc_state[2], cap_inc_nodes[2], cap_inc_reconf, cap_inc_jobs;
    int tile_jobs;                      // job tile of rubick_schedule_round
    int num_sms;
    std::string err;
};

namespace rubick {

int fail(rubick_ctx *ctx, int code, const char *msg);
int cuda_fail(rubick_ctx *ctx, cudaError_t e, const char *what);

// launchers, one per translation unit
cudaError_t launch_eval(const Space &sp, const QuadDesc *d_quads, const void *d_wide_quads, const rubick_job *d_jobs, int J,
                        float *d_thr, uint32_t *d_feas, cudaStream_t st);
cudaError_t launch_curves(const Space &sp, const QuadDesc *d_quads, const void *d_wide_quads, const rubick_job *d_jobs, int J,
                          unsigned flags, uint32_t *d_feas, float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g,
                          cudaStream_t st, int4 *d_top = nullptr);
// d_top (optional, [J][G][C]): the entries at the top memory level once more, packed (value bits, plan, GPUs, 0), for
// the round's preparation, which otherwise has to fetch one 128-byte line per entry from each of the three tables
cudaError_t launch_best(const Space &sp, const float *d_thr, const uint32_t *d_feas, int J, unsigned flags,
                        float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g, uint32_t *d_status,
                        int32_t *d_todo /* J + 1 words of scratch */, int num_sms, cudaStream_t st);
cudaError_t launch_gain(const Space &sp, const rubick_job *d_jobs, int J, const float *d_curve_val,
                        const rubick_assignment *d_state, float *d_gain_gpu, float *d_gain_cpu,
                        int32_t *d_next_g, int32_t *d_next_c, cudaStream_t st);
cudaError_t launch_min_resources(const Space &sp, const QuadDesc *d_quads, const float *d_thr, const uint32_t *d_feas,
                                 const float *d_cv, int J, const rubick_request *d_req, int32_t *d_gmin, int32_t *d_cmin,
                                 float *d_baseline, cudaStream_t st);
cudaError_t launch_fit(const rubick_env &env, const QuadDesc *d_quads, const WideQuad *d_wide_quads, int P, const rubick_job *d_jobs, int J,
                       const rubick_sample *d_samples, int S, int sweeps, double *d_theta, double *d_rmsle, cudaStream_t st);
size_t round_scratch_need(const Space &sp, int J, int N);
size_t incr_scratch_need(const Space &sp, int J, int N);
cudaError_t launch_round_incremental(const Space &sp, const rubick_job *d_jobs, int J, const float *d_cv, const int32_t *d_cp,
                                     const int32_t *d_cg, const uint32_t *d_feas, int N, int max_steps,
                                     const rubick_assignment *d_prev, const rubick_node *d_prev_nodes,
                                     const rubick_reconf *d_reconf, float theta, rubick_assignment *d_out,
                                     rubick_node *d_node_out, int32_t *d_step_log, void *d_scratch,
                                     const int32_t *d_quota, int n_tenants, uint32_t *d_status, int32_t *d_steps,
                                     cudaStream_t st);
cudaError_t launch_round(const Space &sp, const rubick_job *d_jobs, int J, const float *d_cv, const int32_t *d_cp,
                         const int32_t *d_cg, const uint32_t *d_feas, int N, int max_steps,
                         rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                         void *d_scratch, const int32_t *d_quota, int n_tenants,
                         uint32_t *d_status, int32_t *d_steps, cudaStream_t st);

}  // namespace rubick
