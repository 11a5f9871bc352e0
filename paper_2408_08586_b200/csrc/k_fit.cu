// Batched fitting of the performance model (paper Section 4.3, "Continuous model fitting"): for every
// model type, the seven fittable parameters of Table 1 (k_bwd, k_sync, k_opt, k_opt_off, k_off, k_swap,
// k_const) are chosen to minimise the root mean squared logarithmic error between Eq. 1's throughput
// and throughputs measured on sampled (plan, cores) configurations.
//
// The paper names no optimiser; the search here is a pattern search (Hooke and Jeeves) whose every
// decision another implementation can reproduce: start from the coefficients in the job record, clamped
// to fixed bounds; in sweep r move one parameter at a time, in Table 1's order, among base * M^e,
// e = -1, +1, -2, +2, ... +-4 (M = 2^(3/4) at first, its square root after every second sweep), a
// candidate replacing the best so far only if it lowers the squared error by more than one part in 1e9;
// after the sweep repeat its combined displacement (theta^2 / theta_before, element-wise) up to four times
// while that also pays.  Candidate values come from correctly rounded operations only (sqrt, *, /), so
// they are the same numbers in any implementation; only pow / log inside the model may differ in the
// last bits, which matters to a decision only when it sits within rounding of its threshold.
//
// Double precision throughout.  One warp per model: lane q + 8 * part evaluates the q-th of the eight
// candidates of the parameter being moved on the samples i = part (mod 4); the four partial sums of a
// candidate are added pairwise by two shuffles, then every lane walks the eight errors in candidate order.
// The work is a few thousand model evaluations per fit, bound by latency of the FP64 pipe and pow / log.

#include "rubick_internal.cuh"

namespace rubick {

constexpr int FIT_PARAMS = 7;
constexpr int FIT_LANES = 8;          // candidates per parameter move
constexpr int FIT_PARTS = 4;          // lanes that share the samples of one candidate
constexpr double FIT_EPS = 1e-9;

struct FitEnv {
    double B_intra, B_inter, B_pcie, e;
    double z3_volume;                 // factor on V_dp for ZeRO stage 3 (1 = Section 4.1's rule)
    int Gn, strict;
};

__device__ __forceinline__ double overlap(double k, double x, double y)
{
    if (x == 0.0) return y;
    if (y == 0.0) return x;
    return pow(pow(x, k) + pow(y, k), 1.0 / k);
}

// Throughput of Eq. 1 for job jb with trial coefficients th[] under plan `idx` with c cores; 0 when the
// plan is structurally invalid for the job.
__device__ double model_thr(const rubick_job &jb, const double *th, const FitEnv &ev, const QuadDesc *__restrict__ quads,
                            const WideQuad *__restrict__ wide, int idx, double c)
{
    const QuadDesc q = quads[idx >> 2];
    const int v = idx & 3, gc = v >> 1, off = v & 1, z = q.zero;
    if (q.disabled & (1u << v)) return 0.0;
    long long d = 1ll << q.log2d, t = 1ll << q.log2t, p = 1ll << q.log2p;
    int accum = 0;
    if (wide) {                         // degrees of any size and the accumulation setting
        const WideQuad w = wide[idx >> 2];
        d = w.x & 0xffff; t = w.x >> 16; p = w.y & 0xffff; accum = int(w.y >> 24);
    }
    const long long b = jb.b, l = jb.l, h = jb.h;
    if (t > ev.Gn || p > l || d > b || b % d != 0 || (off && z < 2) || h % t != 0) return 0.0;
    if (ev.strict && (z > 0 || off) && (t > 1 || p > 1)) return 0.0;

    const long long r = b / d;
    const long long mu_most = r < jb.mu_cap ? r : jb.mu_cap;
    if ((mu_most >> accum) < 1) return 0.0;
    const long long mu_i = mu_most >> accum;
    const long long n = (r + mu_i - 1) / mu_i;
    const double mu = double(mu_i), m = p > 1 ? double(n) : 1.0, a = p > 1 ? 1.0 : double(n);
    const double dd = double(d), tt = double(t), pp = double(p), g = dd * tt * pp;
    const double P = jb.P, bb = double(b), s = double(jb.s), hh = double(h), ll = double(l);

    double T_fwd = double(jb.tau) * mu / (tt * pp);
    if (p > 1) T_fwd *= (m + pp - 1.0);
    const double T_bwd = th[0] * T_fwd + (gc ? T_fwd : 0.0);

    double V_dp = 0.0, V_tp = 0.0, V_pp = 0.0;
    if (d > 1) V_dp = ev.e * P * 2.0 * (dd - 1.0) / (dd * tt * pp) * (z == 3 ? ev.z3_volume : 1.0);
    if (t > 1) V_tp = ev.e * 4.0 * 2.0 * (tt - 1.0) * bb * s * hh * ll / (dd * tt);
    if (p > 1) V_pp = ev.e * 2.0 * pp * bb * s * hh / (dd * tt);
    const double B_dp = (dd * tt <= double(ev.Gn)) ? ev.B_intra : ev.B_inter;
    const double B_pp = (g <= double(ev.Gn)) ? ev.B_intra : ev.B_inter;
    const double T_dp = V_dp / B_dp, T_tp = V_tp / ev.B_intra, T_pp = V_pp / B_pp;

    const double T_cc = a * T_fwd + (a - 1.0) * T_bwd + overlap(th[1], T_bwd, T_dp) + T_tp + T_pp;
    const double Psi = P / (tt * pp);
    double T_oo;
    if (off) {
        const double T_opt = th[3] * Psi / (dd * c);
        const double T_off = ev.e * Psi / (dd * ev.B_pcie);
        T_oo = overlap(th[4], T_dp, T_off) + overlap(th[5], T_opt, T_off);
    } else {
        T_oo = th[2] * Psi / (z >= 1 ? dd : 1.0);
    }
    const double T_iter = T_cc + T_oo + th[6];
    return bb / T_iter;
}

// Sum of squared log errors over all samples; the lanes that differ only in `part` hold the same th[] and
// end up with the same total (pairwise sums of their partial sums).  Warp-wide.
__device__ double sum_sq_log_err(const rubick_job &jb, const double *th, const FitEnv &ev, const QuadDesc *__restrict__ quads,
                                 const WideQuad *__restrict__ wide, const rubick_sample *__restrict__ smp, int S, int P,
                                 int part, int *n_out)
{
    double sse = 0.0; int n = 0;
    for (int i = part; i < S; i += FIT_PARTS) {
        const rubick_sample x = smp[i];
        if (x.plan < 0 || x.plan >= P) continue;
        const double e = log1p(model_thr(jb, th, ev, quads, wide, x.plan, double(x.cores))) - log1p(x.thr);
        sse += e * e; ++n;
    }
    sse += __shfl_xor_sync(0xffffffffu, sse, 8);
    sse += __shfl_xor_sync(0xffffffffu, sse, 16);
    if (n_out) { n += __shfl_xor_sync(0xffffffffu, n, 8); n += __shfl_xor_sync(0xffffffffu, n, 16); *n_out = n; }
    return sse;
}

__global__ void __launch_bounds__(64)
fit_models_kernel(const __grid_constant__ FitEnv ev, const QuadDesc *__restrict__ quads, const WideQuad *__restrict__ wide, int P,
                  const rubick_job *__restrict__ jobs, int J, const rubick_sample *__restrict__ samples, int S,
                  int sweeps, double *__restrict__ theta_out, double *__restrict__ rmsle_out)
{
    const double lo[FIT_PARAMS] = {0.25, 1.0, 1e-13, 1e-10, 1.0, 1.0, 1e-4};
    const double hi[FIT_PARAMS] = {16.0, 16.0, 1e-9, 1e-6, 16.0, 16.0, 10.0};
    const int lane = threadIdx.x & 31;
    const int q = lane & (FIT_LANES - 1);                       // candidate this lane evaluates
    const int part = lane >> 3;                                 // its share of the samples
    const int j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const bool live = j < J;
    const int jj = live ? j : 0;
    const rubick_job jb = jobs[jj];
    const rubick_sample *smp = samples + size_t(jj) * S;

    double th[FIT_PARAMS] = {double(jb.k_bwd), double(jb.k_sync), double(jb.k_opt), double(jb.k_opt_off),
                             double(jb.k_off), double(jb.k_swap), double(jb.k_const)};
#pragma unroll
    for (int p = 0; p < FIT_PARAMS; ++p) {
        if (!(th[p] >= lo[p])) th[p] = lo[p];
        if (th[p] > hi[p]) th[p] = hi[p];
    }
    int n = 0;
    double cur = sum_sq_log_err(jb, th, ev, quads, wide, smp, S, P, part, &n);
    const double rmsle0 = n > 0 ? sqrt(cur / n) : 0.0;
    double M = sqrt(2.0) * sqrt(sqrt(2.0));
    const int e_of_q = (q & 1) ? ((q >> 1) + 1) : -((q >> 1) + 1);     // q = 0..7 -> -1, +1, -2, +2, -3, +3, -4, +4

    for (int r = 0; r < sweeps; ++r) {
        double mul[5]; mul[0] = 1.0; mul[1] = M; mul[2] = M * M; mul[3] = mul[2] * M; mul[4] = mul[2] * mul[2];
        double before[FIT_PARAMS];
#pragma unroll
        for (int p = 0; p < FIT_PARAMS; ++p) before[p] = th[p];
#pragma unroll
        for (int p = 0; p < FIT_PARAMS; ++p) {
            // every lane of the group tries its own candidate of parameter p
            const double base = th[p];
            double v = e_of_q > 0 ? base * mul[e_of_q] : base / mul[-e_of_q];
            if (v < lo[p]) v = lo[p];
            if (v > hi[p]) v = hi[p];
            th[p] = v;
            const double sse = sum_sq_log_err(jb, th, ev, quads, wide, smp, S, P, part, nullptr);
            th[p] = base;
            // the eight errors in candidate order, as one after the other would see them
            double best = cur, best_v = base;
#pragma unroll
            for (int k = 0; k < FIT_LANES; ++k) {
                const double vk = __shfl_sync(0xffffffffu, v, k);
                const double sk = __shfl_sync(0xffffffffu, sse, k);
                if (vk != base && n > 0 && sk < best * (1.0 - FIT_EPS)) { best = sk; best_v = vk; }
            }
            th[p] = best_v; cur = best;
        }
        // pattern moves: every lane computes the same thing on its share of the samples
        for (int rep = 0; rep < 4 && n > 0; ++rep) {        // (uniform over the warp: all lanes hold the same th and cur)
            double keep[FIT_PARAMS]; bool moved = false;
#pragma unroll
            for (int p = 0; p < FIT_PARAMS; ++p) {
                keep[p] = th[p];
                double v = keep[p] * keep[p] / before[p];
                if (v < lo[p]) v = lo[p];
                if (v > hi[p]) v = hi[p];
                moved |= v != keep[p];
                th[p] = v;
            }
            if (!moved) break;
            const double sse = sum_sq_log_err(jb, th, ev, quads, wide, smp, S, P, part, nullptr);
            if (sse < cur * (1.0 - FIT_EPS)) {
                cur = sse;
#pragma unroll
                for (int p = 0; p < FIT_PARAMS; ++p) before[p] = keep[p];
            } else {
#pragma unroll
                for (int p = 0; p < FIT_PARAMS; ++p) th[p] = keep[p];
                break;
            }
        }
        if (r & 1) M = sqrt(M);
    }
    if (live && lane == 0) {
#pragma unroll
        for (int p = 0; p < FIT_PARAMS; ++p) theta_out[size_t(j) * FIT_PARAMS + p] = th[p];
        rmsle_out[2 * size_t(j)] = rmsle0;
        rmsle_out[2 * size_t(j) + 1] = n > 0 ? sqrt(cur / n) : 0.0;
    }
}

cudaError_t launch_fit(const rubick_env &env, const QuadDesc *d_quads, const WideQuad *d_wide_quads, int P, const rubick_job *d_jobs, int J,
                       const rubick_sample *d_samples, int S, int sweeps, double *d_theta, double *d_rmsle, cudaStream_t st)
{
    if (J == 0) return cudaSuccess;
    FitEnv ev;
    ev.B_intra = env.B_intra; ev.B_inter = env.B_inter; ev.B_pcie = env.B_pcie; ev.e = double(env.bytes_per_elem);
    ev.Gn = env.gpus_per_node; ev.strict = env.strict_zero_dp_only ? 1 : 0; ev.z3_volume = env.zero3_extra_volume ? 1.5 : 1.0;
    const int threads = 64, per_block = threads / 32;
    fit_models_kernel<<<(J + per_block - 1) / per_block, threads, 0, st>>>(ev, d_quads, d_wide_quads, P, d_jobs, J, d_samples, S, sweeps, d_theta, d_rmsle); count_launch();
    return cudaGetLastError();
}

}  // namespace rubick
