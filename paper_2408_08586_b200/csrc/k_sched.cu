// Marginal gains and the greedy scheduling round (paper Section 5.2, Algorithm 1 in
// marginal-gain form).
//
// Gain ("slope") of a job = weighted curve gain per unit of added resource: for GPUs up to the
// smallest level whose curve value strictly exceeds what the job has now, for CPU cores up to
// the next core level, both read at the top host-memory level (memory is not searched, it is
// allocated once the plan is known).  Gains are computed in single precision with one rounding
// per operation (__fmul_rn / __fsub_rn / __fdiv_rn, never fused), so that any other
// implementation of the same arithmetic reaches bit-identical decisions.
//
// The round is inherently sequential (every commit changes node capacities and one job's
// gains), so it runs as ONE persistent CTA that keeps the cluster state and the per-job scan
// state in shared memory and never returns to the host between increments:
//   per step:  (1) all warps rebuild the first-fit table  node(g level, c level)  and the count of
//                  empty nodes;
//              (2) all threads scan their jobs: a candidate counts only if it can be placed;
//              (3) block-wide argmax on a 64-bit key (gain bits << 32 | ~job), GPU gains before
//                  CPU gains;
//              (4) warp 0 commits the winner: placement, host-memory level, curve lookup
//                  (GetBestPlan), memory of that plan (AllocMem), node bookkeeping, new gains.
// The step count is bounded by max_steps; hitting it sets a status bit instead of spinning.

#include <atomic>
#include "round_plain.cuh"

namespace rubick {

__global__ void marginal_gain_kernel(const __grid_constant__ Space sp, const rubick_job *__restrict__ jobs, int J,
                                     const float *__restrict__ cv, const rubick_assignment *__restrict__ state,
                                     float *__restrict__ gain_gpu, float *__restrict__ gain_cpu,
                                     int32_t *__restrict__ next_g, int32_t *__restrict__ next_c)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= J) return;
    const rubick_assignment s = state[j];
    int gi = -1, ci = jobs[j].cmin_idx > 0 ? jobs[j].cmin_idx : 0;
    if (s.g > 0) { gi = level_of_g(sp, s.g); ci = level_of_c(sp, s.c); }
    Gains r;
    if (s.g > 0 && (gi < 0 || ci < 0)) { r.next_g = r.next_c = -1; r.gain_g = r.gain_c = 0.0f; }   // not on the grid
    else r = job_gains(sp, cv, j, jobs[j].w, gi, min(ci, sp.nC - 1), s.thr);
    gain_gpu[j] = r.gain_g; gain_cpu[j] = r.gain_c; next_g[j] = r.next_g; next_c[j] = r.next_c;
}

cudaError_t launch_gain(const Space &sp, const rubick_job *d_jobs, int J, const float *d_curve_val,
                        const rubick_assignment *d_state, float *d_gain_gpu, float *d_gain_cpu,
                        int32_t *d_next_g, int32_t *d_next_c, cudaStream_t st)
{
    if (J == 0) return cudaSuccess;
    marginal_gain_kernel<<<(J + 127) / 128, 128, 0, st>>>(sp, d_jobs, J, d_curve_val, d_state, d_gain_gpu,
                                                         d_gain_cpu, d_next_g, d_next_c); count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// minimum demand of guaranteed jobs (paper Section 5.2): one thread per job walks the curve from the
// smallest allocation upwards, GPUs before cores, and stops at the first one that runs and reaches
// the performance the original plan predicts at the requested resources
// ------------------------------------------------------------------------------------------------
__global__ void min_resources_kernel(const __grid_constant__ Space sp, const QuadDesc *__restrict__ quads,
                                     const float *__restrict__ thr, const uint32_t *__restrict__ feas,
                                     const float *__restrict__ cv, int J, const rubick_request *__restrict__ req,
                                     int32_t *__restrict__ gmin_idx, int32_t *__restrict__ cmin_idx,
                                     float *__restrict__ baseline)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= J) return;
    const rubick_request r = req[j];
    int gm = -1, cm = -1; float base = 0.0f;
    if (r.plan >= 0 && r.plan < sp.P && r.g_idx >= 0 && r.g_idx < sp.nG && r.c_idx >= 0 && r.c_idx < sp.nC
        && r.m_idx >= 0 && r.m_idx < sp.nM) {
        // the original plan runs at the request if it uses exactly that many GPUs and fits that much memory
        const bool runs = quads[r.plan >> 2].g_level == r.g_idx && ((feas[size_t(j) * sp.P + r.plan] >> r.m_idx) & 1u);
        if (runs) base = thr[(size_t(j) * sp.nC + r.c_idx) * sp.P + r.plan];
        gm = r.g_idx; cm = r.c_idx;
        bool found = false;
        for (int gi = 0; gi <= r.g_idx && !found; ++gi)
            for (int ci = 0; ci <= r.c_idx && !found; ++ci) {
                const float v = cv[curve_idx(sp, j, gi, ci, r.m_idx)];
                if (v > 0.0f && v >= base) { gm = gi; cm = ci; found = true; }
            }
    }
    gmin_idx[j] = gm; cmin_idx[j] = cm; baseline[j] = base;
}

cudaError_t launch_min_resources(const Space &sp, const QuadDesc *d_quads, const float *d_thr, const uint32_t *d_feas,
                                 const float *d_cv, int J, const rubick_request *d_req, int32_t *d_gmin, int32_t *d_cmin,
                                 float *d_baseline, cudaStream_t st)
{
    if (J == 0) return cudaSuccess;
    min_resources_kernel<<<(J + 127) / 128, 128, 0, st>>>(sp, d_quads, d_thr, d_feas, d_cv, J, d_req, d_gmin, d_cmin, d_baseline); count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// greedy round
// ------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(ROUND_THREADS, 1)
greedy_round_kernel(const __grid_constant__ Space sp, const rubick_job *__restrict__ jobs, int J,
                    const float *__restrict__ cv, const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                    const uint32_t *__restrict__ feas, int N, int max_steps, rubick_assignment *__restrict__ out,
                    rubick_node *__restrict__ node_out, int32_t *__restrict__ step_log, HotA *hotA_g, HotB *hotB_g,
                    int hot_in_smem, const int32_t *__restrict__ quota, int n_tenants,
                    uint32_t *__restrict__ status, int32_t *__restrict__ steps_out)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ RoundShared sh;
    __shared__ int32_t rem_q[2 * RUBICK_MAX_TENANTS];      // what is left of every tenant's quota: GPUs, cores

    // shared layout: free_m [N] i64 | free_g [N] | free_c [N] | owner [N] | ff [n_small * nC] | hot arrays
    Cluster cl;
    cl.N = N;
    cl.free_m = reinterpret_cast<int64_t *>(smem_raw);
    cl.free_g = reinterpret_cast<int32_t *>(cl.free_m + N);
    cl.free_c = cl.free_g + N;
    cl.owner = cl.free_c + N;
    cl.ff = cl.owner + N;
    const int n_ff = sp.n_small * sp.nC;
    size_t off = size_t(N) * 20 + size_t(n_ff) * 4;
    off = (off + 15) & ~size_t(15);
    HotA *hotA = hot_in_smem ? reinterpret_cast<HotA *>(smem_raw + off) : hotA_g;
    HotB *hotB = hot_in_smem ? reinterpret_cast<HotB *>(smem_raw + off + size_t(J) * sizeof(HotA)) : hotB_g;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mt = sp.nM - 1;

    for (int n = tid; n < N; n += ROUND_THREADS) {
        cl.free_g[n] = sp.Gn; cl.free_c[n] = sp.Cn; cl.free_m[n] = sp.Mn; cl.owner[n] = -1;
    }
    for (int j = tid; j < J; j += ROUND_THREADS) {
        const rubick_job *jb = jobs + j;
        const int gmin = jb->gmin_idx;
        const int c0 = min(max(jb->cmin_idx, 0), sp.nC - 1);
        HotA a; a.gain_g = 0.0f; a.gain_c = 0.0f; a.node = -1;
        a.packed = pack(-1, c0, -1, gmin >= 0, false, false);
        HotB b; b.val = 0.0f; b.plan = -1; b.f_level = -1; b.w = jb->w;
        hotA[j] = a; hotB[j] = b;
    }
    if (tid == 0) { sh.steps = 0; sh.capped = 0; sh.n_empty = N; }
    for (int i = tid; i < 2 * n_tenants; i += ROUND_THREADS) rem_q[i] = quota[i];
    __syncthreads();

    // ---- Phase A: guaranteed minima, in job order (warp 0) ----------------------------------------
    if (warp == 0) {
        int n_empty = N;
        for (int base = 0; base < J; base += 32) {
            const int jj = base + lane;
            const bool want = jj < J && pk_pending(hotA[jj].packed);
            unsigned todo = __ballot_sync(0xffffffffu, want);
            while (todo) {
                const int j = base + __ffs(todo) - 1;
                todo &= todo - 1;
                const rubick_job *jb = jobs + j;
                const int gmin = jb->gmin_idx, cmin = max(jb->cmin_idx, 0);
                if (gmin >= sp.nG || cmin >= sp.nC) continue;
                const size_t o = curve_idx(sp, j, gmin, cmin, mt);
                if (__ldg(cp + o) < 0) continue;
                // the curve may reach this value with fewer GPUs than the level offers
                const int gi = level_of_g(sp, __ldg(cg + o));
                if (gi < 0) continue;
                const int tn = jb->tenant;
                if (n_tenants > 0) {       // privileged only while the minimum fits the tenant's remaining quota
                    if (tn < 0 || tn >= n_tenants) continue;
                    if (rem_q[2 * tn] < sp.g_levels[gi] || rem_q[2 * tn + 1] < sp.c_levels[cmin]) continue;
                }
                HotA a = hotA[j]; HotB b = hotB[j];
                if (commit_warp(sp, cl, n_empty, cv, cp, cg, feas, j, a, b, gi, cmin, false, lane)) {
                    if (lane == 0) { hotA[j] = a; hotB[j] = b; }
                    if (lane == 0 && n_tenants > 0) { rem_q[2 * tn] -= sp.g_levels[gi]; rem_q[2 * tn + 1] -= sp.c_levels[cmin]; }
                    __syncwarp();
                    // recount empty nodes
                    int cnt = 0;
                    for (int nb = 0; nb < N; nb += 32) {
                        const int n = nb + lane;
                        cnt += __popc(__ballot_sync(0xffffffffu, n < N && cl.free_g[n] == sp.Gn));
                    }
                    n_empty = cnt;
                }
                __syncwarp();
            }
        }
    }
    __syncthreads();

    // initial gains of every job that may still grow
    for (int j = tid; j < J; j += ROUND_THREADS) {
        HotA a = hotA[j];
        if (pk_pending(a.packed)) continue;
        const Gains r = job_gains(sp, cv, j, hotB[j].w, pk_gi(a.packed), pk_ci(a.packed), hotB[j].val);
        a.gain_g = r.gain_g; a.gain_c = r.gain_c;
        a.packed = pack(pk_gi(a.packed), pk_ci(a.packed), r.next_g, false, false, false);
        hotA[j] = a;
    }
    __syncthreads();

    // ---- Phase B: greedy increments -----------------------------------------------------------------
    for (;;) {
        // (1) first-fit table and empty-node count
        for (int e = warp; e <= n_ff; e += ROUND_WARPS) {
            if (e == n_ff) {
                int cnt = 0;
                for (int nb = 0; nb < N; nb += 32) {
                    const int n = nb + lane;
                    cnt += __popc(__ballot_sync(0xffffffffu, n < N && cl.free_g[n] == sp.Gn));
                }
                if (lane == 0) sh.n_empty = cnt;
            } else {
                const int gi = e / sp.nC, ci = e - gi * sp.nC;
                const int n = first_fit_warp(cl, sp.g_levels[gi], sp.c_levels[ci], lane);
                if (lane == 0) cl.ff[e] = n;
            }
        }
        __syncthreads();

        // (2) scan: best placeable GPU increment and best placeable CPU increment of my jobs
        const int n_empty = sh.n_empty;
        unsigned long long best_g = 0ull, best_c = 0ull;
        for (int j = tid; j < J; j += ROUND_THREADS) {
            const HotA a = hotA[j];
            const unsigned long long kg = (static_cast<unsigned long long>(__float_as_uint(a.gain_g)) << 32) | (0xffffffffu - uint32_t(j));
            const unsigned long long kc = (static_cast<unsigned long long>(__float_as_uint(a.gain_c)) << 32) | (0xffffffffu - uint32_t(j));
            const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
            if (a.gain_g > 0.0f && kg > best_g && placeable(sp, cl, n_empty, gi, ci, a.node, pk_next_gi(a.packed), ci)) best_g = kg;
            if (a.gain_c > 0.0f && kc > best_c && placeable(sp, cl, n_empty, gi, ci, a.node, gi, ci + 1)) best_c = kc;
        }
        // (3) block argmax
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
            const unsigned long long og = __shfl_xor_sync(0xffffffffu, best_g, s);
            const unsigned long long oc = __shfl_xor_sync(0xffffffffu, best_c, s);
            best_g = og > best_g ? og : best_g;
            best_c = oc > best_c ? oc : best_c;
        }
        if (lane == 0) { sh.red[0][warp] = best_g; sh.red[1][warp] = best_c; }
        __syncthreads();
        if (warp == 0) {
            unsigned long long bg = sh.red[0][lane], bc = sh.red[1][lane];
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) {
                const unsigned long long og = __shfl_xor_sync(0xffffffffu, bg, s);
                const unsigned long long oc = __shfl_xor_sync(0xffffffffu, bc, s);
                bg = og > bg ? og : bg;
                bc = oc > bc ? oc : bc;
            }
            int sel_j = -1, sel_type = -1;
            if (bg) { sel_j = int(0xffffffffu - uint32_t(bg)); sel_type = 0; }
            else if (bc) { sel_j = int(0xffffffffu - uint32_t(bc)); sel_type = 1; }
            if (sel_j >= 0 && sh.steps >= max_steps) { if (lane == 0) sh.capped = 1; sel_j = -1; }

            // (4) commit
            if (sel_j >= 0) {
                const int j = sel_j;
                HotA a = hotA[j]; HotB b = hotB[j];
                const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
                const int gi2 = sel_type == 0 ? pk_next_gi(a.packed) : gi;
                const int ci2 = sel_type == 0 ? ci : ci + 1;
                const bool ok = commit_warp(sp, cl, n_empty, cv, cp, cg, feas, j, a, b, gi2, ci2, true, lane);
                bool fz_g = pk_fz_g(a.packed), fz_c = pk_fz_c(a.packed);
                if (!ok) { if (sel_type == 0) fz_g = true; else fz_c = true; }
                const Gains r = job_gains(sp, cv, j, b.w, pk_gi(a.packed), pk_ci(a.packed), b.val);
                a.gain_g = fz_g ? 0.0f : r.gain_g;
                a.gain_c = fz_c ? 0.0f : r.gain_c;
                a.packed = pack(pk_gi(a.packed), pk_ci(a.packed), r.next_g, false, fz_g, fz_c);
                if (lane == 0) {
                    hotA[j] = a; hotB[j] = b;
                    if (step_log) step_log[sh.steps] = (j << 2) | (sel_type << 1) | int(ok);
                    sh.steps += 1;
                }
            }
            if (lane == 0) sh.sel_j = sel_j;
        }
        __syncthreads();
        if (sh.sel_j < 0) break;
    }

    // ---- results ------------------------------------------------------------------------------------
    for (int j = tid; j < J; j += ROUND_THREADS) {
        const HotA a = hotA[j]; const HotB b = hotB[j];
        const int gi = pk_gi(a.packed);
        rubick_assignment r;
        if (gi >= 0) {
            r.g = sp.g_levels[gi]; r.c = sp.c_levels[pk_ci(a.packed)]; r.m_bytes = sp.m_levels[b.f_level];
            r.plan = b.plan; r.first_node = a.node; r.n_nodes = max(r.g >> sp.log2Gn, 1);
            r.thr = b.val; r.status = RUBICK_RUNNING; r.m_level = b.f_level;
        } else {
            r.g = 0; r.c = 0; r.m_bytes = 0; r.plan = -1; r.first_node = -1; r.n_nodes = 0; r.thr = 0.0f;
            r.status = pk_pending(a.packed) ? RUBICK_PENDING : RUBICK_UNALLOCATED; r.m_level = -1;
        }
        out[j] = r;
    }
    if (node_out)
        for (int n = tid; n < N; n += ROUND_THREADS) {
            rubick_node nd;
            nd.free_g = cl.free_g[n]; nd.free_c = cl.free_c[n]; nd.free_m = cl.free_m[n]; nd.owner = cl.owner[n];
            nd.reserved = 0;
            node_out[n] = nd;
        }
    if (tid == 0) {
        *steps_out = sh.steps;
        if (sh.capped) atomicOr(status, DS_STEP_CAP);
    }
}

static size_t round_fixed_smem(const Space &sp, int N)
{
    size_t off = size_t(N) * 20 + size_t(sp.n_small) * sp.nC * 4;
    return (off + 15) & ~size_t(15);
}
constexpr size_t ROUND_SMEM_LIMIT = 200 * 1024;

static bool hot_fits_smem(const Space &sp, int J, int N)
{
    return round_fixed_smem(sp, N) + size_t(J) * (sizeof(HotA) + sizeof(HotB)) <= ROUND_SMEM_LIMIT;
}

size_t round_scratch_need(const Space &sp, int J, int N)
{
    return hot_fits_smem(sp, J, N) ? 0 : size_t(J) * (sizeof(HotA) + sizeof(HotB));
}

cudaError_t launch_round(const Space &sp, const rubick_job *d_jobs, int J, const float *d_cv, const int32_t *d_cp,
                         const int32_t *d_cg, const uint32_t *d_feas, int N, int max_steps,
                         rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                         void *d_scratch, const int32_t *d_quota, int n_tenants,
                         uint32_t *d_status, int32_t *d_steps, cudaStream_t st)
{
    // every step either raises one job by a level or freezes one (job, resource) pair, so a
    // round cannot take more steps than this; the clamp keeps the device loop bounded regardless
    const long long natural = (long long)J * (sp.nG + sp.nC + 2) + 1;
    if ((long long)max_steps > natural) max_steps = int(natural < 0x7fffffffLL ? natural : 0x7fffffffLL);
    const bool in_smem = hot_fits_smem(sp, J, N);
    const size_t smem = round_fixed_smem(sp, N) + (in_smem ? size_t(J) * (sizeof(HotA) + sizeof(HotB)) : 0);
    cudaError_t e = cudaFuncSetAttribute(greedy_round_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(ROUND_SMEM_LIMIT));
    if (e != cudaSuccess) return e;
    HotA *ha = reinterpret_cast<HotA *>(d_scratch);
    HotB *hb = reinterpret_cast<HotB *>(reinterpret_cast<unsigned char *>(d_scratch) + size_t(J) * sizeof(HotA));
    greedy_round_kernel<<<1, ROUND_THREADS, smem, st>>>(sp, d_jobs, J, d_cv, d_cp, d_cg, d_feas, N, max_steps, d_out,
                                                        d_node_out, d_step_log, ha, hb, in_smem ? 1 : 0, d_quota, n_tenants,
                                                        d_status, d_steps); count_launch();
    return cudaGetLastError();
}

}  // namespace rubick

// ------------------------------------------------------------------------------------------------
// Greedy round for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc when they schedule: a scheduler daemon that
// was given a fixed device-memory budget at start-up and shares the GPU with jobs that fill the
// rest of it (a late allocation may fail, and it synchronises the whole device while it runs), or
// a process whose device memory is owned by a framework's caching allocator that has already
// reserved everything.  rubick_greedy_round grows a context scratch buffer with cudaMalloc when
// the per-job scan state does not fit shared memory; the entry point below never allocates: the
// per-job state always lives in the fixed array declared here, which every GPU that loads the
// library holds until the process exits.
// ------------------------------------------------------------------------------------------------

namespace rubick {

constexpr size_t NOALLOC_STATE_BYTES = size_t(RUBICK_NOALLOC_MAX_JOBS) * (sizeof(HotA) + sizeof(HotB));   // 1 MiB
static __device__ __align__(256) unsigned char g_noalloc_state[NOALLOC_STATE_BYTES];

// In host code `g_noalloc_state` is only a handle; the device address has to be asked for, once
// per device, with that device current.  The answer is kept for the life of the process (atomic: two
// host threads making their first call on a device both store the same address).  It refers to the
// device's primary context: after a cudaDeviceReset of that device the stored address is stale, so a
// process that resets a device must not call this entry point on it afterwards.
constexpr int NOALLOC_MAX_DEVICES = 64;
static std::atomic<void *> g_noalloc_addr[NOALLOC_MAX_DEVICES];

}  // namespace rubick

extern "C" int rubick_greedy_round_noalloc(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                                           const float *d_curve_val, const int32_t *d_curve_plan,
                                           const int32_t *d_curve_g, const uint32_t *d_feas,
                                           const rubick_cluster *h_cluster, int max_steps,
                                           rubick_assignment *d_out, rubick_node *d_node_out, int32_t *h_steps)
{
    using namespace rubick;
    if (!ctx) return RUBICK_EINVAL;
    if (!ctx->has_space) return fail(ctx, RUBICK_ESTATE, "no plan space: call rubick_set_space first");
    if (J < 0 || max_steps < 0) return fail(ctx, RUBICK_EINVAL, "negative job count or max_steps");
    if (J > RUBICK_NOALLOC_MAX_JOBS)
        return fail(ctx, RUBICK_EINVAL, "rubick_greedy_round_noalloc: more than RUBICK_NOALLOC_MAX_JOBS jobs; the fixed state array cannot hold them");
    if (!h_cluster || h_cluster->n_nodes < 1 || h_cluster->n_nodes > RUBICK_MAX_NODES)
        return fail(ctx, RUBICK_EINVAL, "cluster: 1 .. RUBICK_MAX_NODES nodes");
    if (h_cluster->n_tenants != 0) return fail(ctx, RUBICK_EINVAL, "rubick_greedy_round_noalloc: tenant quotas are not supported (n_tenants must be 0)");
    if (J > 0 && (!d_jobs || !d_curve_val || !d_curve_plan || !d_curve_g || !d_feas || !d_out))
        return fail(ctx, RUBICK_EINVAL, "null pointer");
    if (ctx->device < 0 || ctx->device >= NOALLOC_MAX_DEVICES) return fail(ctx, RUBICK_EINVAL, "device index out of range");
    const Space &sp = ctx->space;
    const int N = h_cluster->n_nodes;
    const size_t smem = round_fixed_smem(sp, N);
    if (smem > ROUND_SMEM_LIMIT) return fail(ctx, RUBICK_EINVAL, "cluster state does not fit shared memory");

    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaSetDevice");
    void *addr = g_noalloc_addr[ctx->device].load(std::memory_order_acquire);
    if (!addr) {                                 // first call on this device: resolve the array's device address
        e = cudaGetSymbolAddress(&addr, g_noalloc_state);
        if (e != cudaSuccess || !addr) return cuda_fail(ctx, e, "cudaGetSymbolAddress (fixed round state)");
        g_noalloc_addr[ctx->device].store(addr, std::memory_order_release);
    }
    unsigned char *base = static_cast<unsigned char *>(addr);
    HotA *ha = reinterpret_cast<HotA *>(base);
    HotB *hb = reinterpret_cast<HotB *>(base + size_t(RUBICK_NOALLOC_MAX_JOBS) * sizeof(HotA));

    const long long natural = (long long)J * (sp.nG + sp.nC + 2) + 1;
    if ((long long)max_steps > natural) max_steps = int(natural < 0x7fffffffLL ? natural : 0x7fffffffLL);
    e = cudaFuncSetAttribute(greedy_round_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(ROUND_SMEM_LIMIT));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute");
    // the kernel writes every job's state before it reads it, so stale contents of the array
    // from an earlier call need no clearing
    greedy_round_kernel<<<1, ROUND_THREADS, smem, ctx->stream>>>(sp, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas,
                                                                 N, max_steps, d_out, d_node_out, nullptr, ha, hb, 0,
                                                                 nullptr, 0, ctx->d_status, ctx->d_steps); count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch greedy_round (fixed state)");

    uint32_t two[2] = {0u, 0u};
    e = cudaMemcpyAsync(two, ctx->d_status, 8, cudaMemcpyDeviceToHost, ctx->stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "read round status");
    e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaStreamSynchronize");
    if (h_steps) *h_steps = int32_t(two[1]);
    if (two[0] & DS_STEP_CAP) {
        const uint32_t cleared = two[0] & ~uint32_t(DS_STEP_CAP);
        cudaMemcpyAsync(ctx->d_status, &cleared, 4, cudaMemcpyHostToDevice, ctx->stream);
        cudaStreamSynchronize(ctx->stream);
        return fail(ctx, RUBICK_ESTEPS, "greedy round stopped at max_steps");
    }
    return RUBICK_OK;
}
