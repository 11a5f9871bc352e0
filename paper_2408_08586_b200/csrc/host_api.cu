// Host side of librubick: context, plan enumerator, validation and the extern "C" entry points.
// Every entry point validates its arguments, then enqueues kernels on the context's stream.

#include <cstdio>
#include <cstring>
#include <new>

#include "rubick_internal.cuh"

using namespace rubick;

namespace rubick {

int fail(rubick_ctx *ctx, int code, const char *msg)
{
    if (ctx) ctx->err = msg;
    return code;
}

int cuda_fail(rubick_ctx *ctx, cudaError_t e, const char *what)
{
    if (ctx) {
        ctx->err = std::string(what) + ": " + cudaGetErrorString(e);
    }
    // the runtime also remembers a failed call (a refused cudaMalloc, say) as its "last error"; take it out, or the
    // next launch's own error check would report it
    (void)cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? RUBICK_ENOMEM : RUBICK_ECUDA;
}

static bool is_pow2(int64_t x) { return x > 0 && (x & (x - 1)) == 0; }
static int ilog2(int64_t x) { int n = 0; while ((int64_t(1) << (n + 1)) <= x) ++n; return n; }

// grows a device buffer to at least `need` elements (contents are not preserved)
template <typename T>
static int ensure(rubick_ctx *ctx, T *&ptr, size_t &cap, size_t need)
{
    if (need <= cap) return RUBICK_OK;
    if (ptr) { cudaFree(ptr); ptr = nullptr; cap = 0; }
    cudaError_t e = cudaMalloc(reinterpret_cast<void **>(&ptr), need * sizeof(T));
    if (e != cudaSuccess) { ptr = nullptr; return cuda_fail(ctx, e, "cudaMalloc (scratch)"); }
    cap = need;
    return RUBICK_OK;
}

}  // namespace rubick

#define CHECK_CTX(ctx) do { if (!(ctx)) return RUBICK_EINVAL; } while (0)
#define CUDA_TRY(ctx, call, what) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail(ctx, e_, what); } while (0)

extern "C" {

int rubick_create(rubick_ctx **out, const rubick_env *h_env, int device, void *cuda_stream)
{
    if (!out || !h_env) return RUBICK_EINVAL;
    *out = nullptr;
    const rubick_env &e = *h_env;
    if (!(e.B_intra > 0) || !(e.B_inter > 0) || !(e.B_pcie > 0) || e.gpu_mem_bytes <= 0 || e.mem_per_node_bytes <= 0
        || e.gpus_per_node <= 0 || e.cpus_per_node <= 0 || e.bytes_per_elem <= 0 || !is_pow2(e.gpus_per_node))
        return RUBICK_EINVAL;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return RUBICK_ECUDA;
    if (cudaSetDevice(device) != cudaSuccess) return RUBICK_ECUDA;
    rubick_ctx *ctx = new (std::nothrow) rubick_ctx();
    if (!ctx) return RUBICK_ENOMEM;
    ctx->env = e;
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->has_space = false;
    ctx->d_quads = nullptr; ctx->d_wide_quads = nullptr; ctx->d_status = nullptr; ctx->d_steps = nullptr;
    ctx->d_round_scratch = nullptr; ctx->round_scratch_bytes = 0;
    ctx->d_thr = nullptr; ctx->d_feas = nullptr; ctx->d_cv = nullptr; ctx->d_cp = nullptr; ctx->d_cg = nullptr;
    ctx->cap_thr = ctx->cap_feas = ctx->cap_curve = 0;
    ctx->d_top = nullptr; ctx->cap_top = 0;
    ctx->d_jobs_stage = nullptr; ctx->cap_jobs = 0;
    ctx->d_out_stage = nullptr; ctx->cap_out = 0;
    ctx->d_node_stage = nullptr; ctx->cap_node = 0;
    ctx->d_best_todo = nullptr; ctx->cap_best_todo = 0;
    ctx->inc_J = 0; ctx->inc_N = 0; ctx->inc_cur = 0;
    for (int i = 0; i < 2; ++i) { ctx->d_inc_state[i] = nullptr; ctx->d_inc_nodes[i] = nullptr; ctx->cap_inc_state[i] = 0; ctx->cap_inc_nodes[i] = 0; }
    ctx->d_inc_reconf = nullptr; ctx->cap_inc_reconf = 0; ctx->d_inc_jobs = nullptr; ctx->cap_inc_jobs = 0;
    ctx->tile_jobs = 2048;            // 0.5 GB table tile at 2,640 plans x 24 core levels
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return RUBICK_ECUDA; }
    ctx->num_sms = prop.multiProcessorCount;
    if (cudaMalloc(reinterpret_cast<void **>(&ctx->d_status), 8 + 8 * RUBICK_MAX_TENANTS) != cudaSuccess) { delete ctx; return RUBICK_ENOMEM; }
    ctx->d_steps = reinterpret_cast<int32_t *>(ctx->d_status + 1);
    ctx->d_quota = reinterpret_cast<int32_t *>(ctx->d_status + 2);
    if (cudaMemsetAsync(ctx->d_status, 0, 8, ctx->stream) != cudaSuccess) { cudaFree(ctx->d_status); delete ctx; return RUBICK_ECUDA; }
    *out = ctx;
    return RUBICK_OK;
}

void rubick_destroy(rubick_ctx *ctx)
{
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    cudaFree(ctx->d_quads); cudaFree(ctx->d_wide_quads); cudaFree(ctx->d_status); cudaFree(ctx->d_round_scratch);
    cudaFree(ctx->d_thr); cudaFree(ctx->d_feas); cudaFree(ctx->d_cv); cudaFree(ctx->d_cp); cudaFree(ctx->d_cg);
    cudaFree(ctx->d_top);
    cudaFree(ctx->d_jobs_stage); cudaFree(ctx->d_out_stage); cudaFree(ctx->d_node_stage);
    cudaFree(ctx->d_best_todo);
    for (int i = 0; i < 2; ++i) { cudaFree(ctx->d_inc_state[i]); cudaFree(ctx->d_inc_nodes[i]); }
    cudaFree(ctx->d_inc_reconf); cudaFree(ctx->d_inc_jobs);
    delete ctx;
}

const char *rubick_last_error(const rubick_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int rubick_sync(rubick_ctx *ctx)
{
    CHECK_CTX(ctx);
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
    uint32_t st = 0;
    CUDA_TRY(ctx, cudaMemcpy(&st, ctx->d_status, 4, cudaMemcpyDeviceToHost), "read status");
    if (st & DS_FEAS_NOT_THRESHOLD) {
        cudaMemset(ctx->d_status, 0, 4);
        return fail(ctx, RUBICK_ESTATE, "a feasibility word is not a threshold in the memory-level index");
    }
    return RUBICK_OK;
}

int rubick_enumerate_plans(const int32_t *h_g_levels, int nG, rubick_plan *h_out, int cap, int *n_out,
                           int32_t *h_group_off)
{
    if (!h_g_levels || nG < 1 || nG > RUBICK_MAX_G_LEVELS || !n_out || cap < 0 || (cap > 0 && !h_out)) return RUBICK_EINVAL;
    for (int i = 0; i < nG; ++i)
        if (h_g_levels[i] <= 0 || (i && h_g_levels[i] <= h_g_levels[i - 1])) return RUBICK_EINVAL;
    int n = 0;
    for (int gi = 0; gi < nG; ++gi) {
        if (h_group_off) h_group_off[gi] = n;
        const int g = h_g_levels[gi];
        if (!is_pow2(g)) continue;            // only power-of-two GPU counts factor into (d, t, p)
        const int lg = ilog2(g);
        for (int lt = 0; lt <= lg; ++lt)
            for (int lp = 0; lp + lt <= lg; ++lp)
                for (int z = 0; z < 4; ++z)
                    for (int v = 0; v < 4; ++v, ++n)
                        if (n < cap) {
                            rubick_plan &pl = h_out[n];
                            pl.log2d = uint8_t(lg - lt - lp); pl.log2t = uint8_t(lt); pl.log2p = uint8_t(lp);
                            pl.zero = uint8_t(z); pl.gc = uint8_t(v >> 1); pl.off = uint8_t(v & 1);
                            pl.g_level = uint8_t(gi); pl.disabled = 0;
                        }
    }
    if (h_group_off) h_group_off[nG] = n;
    *n_out = n;
    return RUBICK_OK;
}

}  // extern "C"

namespace {

// Quad tables of a plan list for a placement class (align = 0: packed; a > 0: spread in pieces of a GPUs).
// Section 4.1: a group whose GPUs sit on several nodes talks at the inter-node bandwidth.  Packed: a job of at
// most one node's GPUs sits on one node, a larger one on whole nodes (TP fastest, then DP, then PP).  Spread:
// only jobs one node could hold, in at least two pieces; a tensor-parallel group never straddles pieces (t
// divides a), a data-parallel group stays inside a piece only if d * t divides it, pipeline stages of different
// pieces are on different nodes.  Plans that cannot be spread are disabled for the class.
void build_quads(const std::vector<NormPlan> &plans, const int32_t *g_levels, int Gn, bool wide, int align,
                 std::vector<QuadDesc> &quads, std::vector<WideQuad> &wquads)
{
    const size_t Q = plans.size() / 4;
    quads.assign(Q, QuadDesc());
    wquads.assign(wide ? Q : 0, WideQuad());
    for (size_t i = 0; i < plans.size(); ++i) {
        const NormPlan &pl = plans[i];
        const int v = int(i & 3);
        QuadDesc &q = quads[i >> 2];
        if (v == 0) {
            q.log2d = wide ? 0 : uint8_t(ilog2(pl.d)); q.log2t = wide ? 0 : uint8_t(ilog2(pl.t)); q.log2p = wide ? 0 : uint8_t(ilog2(pl.p));
            q.zero = uint8_t(pl.zero); q.g_level = uint8_t(pl.g_level);
            q.flags = 0; q.disabled = 0; q.pad = 0;
            const int64_t d = pl.d, t = pl.t, g = g_levels[pl.g_level];
            if (align == 0) {
                if (t <= Gn) q.flags |= QF_T_FITS_NODE;
                if (d * t > Gn) q.flags |= QF_DP_INTER;
                if (g > Gn) q.flags |= QF_PP_INTER;
            } else {
                const bool may = g <= Gn && g > align && g % align == 0 && align % t == 0;
                if (may) q.flags |= QF_T_FITS_NODE;
                if (align % (d * t) != 0) q.flags |= QF_DP_INTER;
                q.flags |= QF_PP_INTER;
                if (!may) q.disabled = 0xf;
            }
        }
        if (pl.disabled) q.disabled |= uint8_t(1u << v);
    }
    for (size_t i = 0; i < wquads.size(); ++i) {
        const NormPlan &pl = plans[4 * i];
        wquads[i].x = uint32_t(pl.d) | (uint32_t(pl.t) << 16);
        wquads[i].y = uint32_t(pl.p) | (uint32_t(pl.zero) << 16) | (uint32_t(pl.accum) << 24);
        wquads[i].z = uint32_t(quads[i].flags) | (uint32_t(quads[i].disabled) << 8);
        wquads[i].w = 0u;
    }
}

// uploads quad tables beside the old ones and swaps them in only when everything has succeeded
int upload_quads(rubick_ctx *ctx, const std::vector<QuadDesc> &quads, const std::vector<WideQuad> &wquads)
{
    CUDA_TRY(ctx, cudaSetDevice(ctx->device), "cudaSetDevice");
    QuadDesc *new_quads = nullptr;
    WideQuad *new_wide = nullptr;
    cudaError_t ce = cudaMalloc(reinterpret_cast<void **>(&new_quads), quads.size() * sizeof(QuadDesc));
    if (ce == cudaSuccess) ce = cudaMemcpy(new_quads, quads.data(), quads.size() * sizeof(QuadDesc), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess && !wquads.empty()) {
        ce = cudaMalloc(reinterpret_cast<void **>(&new_wide), wquads.size() * sizeof(WideQuad));
        if (ce == cudaSuccess) ce = cudaMemcpy(new_wide, wquads.data(), wquads.size() * sizeof(WideQuad), cudaMemcpyHostToDevice);
    }
    if (ce != cudaSuccess) {
        cudaFree(new_quads); cudaFree(new_wide);
        return cuda_fail(ctx, ce, "plan tables (allocation or upload)");
    }
    cudaStreamSynchronize(ctx->stream);         // kernels of earlier calls may still read the old tables
    cudaFree(ctx->d_quads); cudaFree(ctx->d_wide_quads);
    ctx->d_quads = new_quads; ctx->d_wide_quads = new_wide;
    return RUBICK_OK;
}

int install_space(rubick_ctx *ctx, const NormPlan *h_plans, int P, const rubick_grid *h_grid, bool wide)
{
    if (!h_grid || P <= 0 || (P & 3)) return fail(ctx, RUBICK_EINVAL, "plans: need a positive multiple of 4");
    const rubick_grid &gr = *h_grid;
    if (P > 65520) return fail(ctx, RUBICK_EINVAL, "plans: at most 65,520 plans (per-job plan tables live in shared memory)");
    if (gr.nG < 1 || gr.nG > RUBICK_MAX_G_LEVELS || gr.nC < 1 || gr.nC > RUBICK_MAX_C_LEVELS || gr.nM < 1
        || gr.nM > RUBICK_MAX_M_LEVELS || !gr.g_levels || !gr.c_levels || !gr.m_levels_bytes)
        return fail(ctx, RUBICK_EINVAL, "grid: level counts out of range or null axes");
    const int Gn = ctx->env.gpus_per_node;
    for (int i = 0; i < gr.nG; ++i) {
        const int g = gr.g_levels[i];
        if (g <= 0 || (i && g <= gr.g_levels[i - 1]) || (g > Gn && g % Gn)) return fail(ctx, RUBICK_EINVAL, "grid: GPU levels must increase; levels above a node must be whole nodes");
    }
    for (int i = 0; i < gr.nC; ++i)
        if (gr.c_levels[i] <= 0 || (i && gr.c_levels[i] <= gr.c_levels[i - 1])) return fail(ctx, RUBICK_EINVAL, "grid: CPU levels must be positive and increasing");
    for (int i = 0; i < gr.nM; ++i)
        if (gr.m_levels_bytes[i] <= 0 || (i && gr.m_levels_bytes[i] <= gr.m_levels_bytes[i - 1])) return fail(ctx, RUBICK_EINVAL, "grid: memory levels must be positive and increasing");

    Space sp;
    std::memset(&sp, 0, sizeof sp);
    sp.P = P; sp.Q = P / 4; sp.nG = gr.nG; sp.nC = gr.nC; sp.nM = gr.nM;
    sp.Gn = Gn; sp.log2Gn = ilog2(Gn); sp.Cn = ctx->env.cpus_per_node;
    sp.strict = ctx->env.strict_zero_dp_only ? 1 : 0;
    sp.z3_volume = ctx->env.zero3_extra_volume ? 1.5f : 1.0f;
    sp.wide = wide ? 1 : 0;
    sp.e = float(ctx->env.bytes_per_elem);
    sp.inv_B_intra = float(1.0 / ctx->env.B_intra);
    sp.inv_B_inter = float(1.0 / ctx->env.B_inter);
    sp.inv_B_pcie = float(1.0 / ctx->env.B_pcie);
    sp.gpu_mem = ctx->env.gpu_mem_bytes; sp.Mn = ctx->env.mem_per_node_bytes;
    for (int i = 0; i < gr.nG; ++i) { sp.g_levels[i] = gr.g_levels[i]; if (gr.g_levels[i] <= Gn) sp.n_small = i + 1; }
    for (int i = 0; i < gr.nC; ++i) { sp.c_levels[i] = gr.c_levels[i]; sp.inv_c[i] = 1.0f / float(gr.c_levels[i]); }
    for (int i = 0; i < gr.nM; ++i) sp.m_levels[i] = gr.m_levels_bytes[i];

    // plans: ordered by level, quads of (gc, off), GPU count = the level's
    int level = 0;
    sp.group_off[0] = 0;
    for (int i = 0; i < P; ++i) {
        const NormPlan &pl = h_plans[i];
        if (pl.g_level >= gr.nG || pl.g_level < level) return fail(ctx, RUBICK_EINVAL, "plans: g_level out of range or not ascending");
        if (pl.zero < 0 || pl.zero > 3 || pl.gc < 0 || pl.gc > 1 || pl.off < 0 || pl.off > 1 || pl.d < 1 || pl.t < 1 || pl.p < 1
            || pl.d > 32768 || pl.t > 32768 || pl.p > 32768 || int64_t(pl.d) * pl.t * pl.p > (int64_t(1) << 20)
            || pl.accum < 0 || pl.accum > 30 || (!wide && pl.accum))
            return fail(ctx, RUBICK_EINVAL, "plans: field out of range");
        if (int64_t(pl.d) * pl.t * pl.p != gr.g_levels[pl.g_level])
            return fail(ctx, RUBICK_EINVAL, "plans: d*t*p differs from the GPU level");
        if (!wide && (!is_pow2(pl.d) || !is_pow2(pl.t) || !is_pow2(pl.p)))
            return fail(ctx, RUBICK_EINVAL, "plans: degrees must be powers of two in this plan format");
        if (pl.g_level > level) {
            if (i & 3) return fail(ctx, RUBICK_EINVAL, "plans: a level must start on a quad boundary");
            while (level < pl.g_level) sp.group_off[++level] = i;
        }
        const int v = i & 3;
        if (pl.gc != (v >> 1) || pl.off != (v & 1)) return fail(ctx, RUBICK_EINVAL, "plans: quads must run (gc, off) = (0,0), (0,1), (1,0), (1,1)");
        if (v != 0) {
            const NormPlan &first = h_plans[i - v];
            if (first.d != pl.d || first.t != pl.t || first.p != pl.p || first.zero != pl.zero || first.accum != pl.accum)
                return fail(ctx, RUBICK_EINVAL, "plans: the four plans of a quad must share d, t, p and the ZeRO stage");
        }
    }
    // four consecutive quads = ZeRO stages 0..3 of one (d, t, p) triple (the evaluation kernel's lanes rely on it)
    if ((P / 4) % 4) return fail(ctx, RUBICK_EINVAL, "plans: every (d, t, p) must come with all four ZeRO stages");
    for (int i = 0; i < P / 4; ++i) {
        const NormPlan &pa = h_plans[4 * (i & ~3)], &pb = h_plans[4 * i];
        if (pb.zero != (i & 3) || pa.d != pb.d || pa.t != pb.t || pa.p != pb.p || pa.accum != pb.accum || pa.g_level != pb.g_level)
            return fail(ctx, RUBICK_EINVAL, "plans: every (d, t, p) must come with ZeRO stages 0..3 in order (disable plans instead of dropping them)");
    }
    while (level < gr.nG) sp.group_off[++level] = P;
    std::vector<NormPlan> kept(h_plans, h_plans + P);
    std::vector<QuadDesc> quads;
    std::vector<WideQuad> wquads;
    build_quads(kept, sp.g_levels, Gn, wide, 0, quads, wquads);
    int rc = upload_quads(ctx, quads, wquads);
    if (rc) return rc;
    ctx->norm_plans.swap(kept);
    ctx->placement_align = 0;
    ctx->space = sp;
    ctx->inc_J = 0;
    ctx->has_space = true;
    return RUBICK_OK;
}


}  // namespace

extern "C" {

int rubick_set_space(rubick_ctx *ctx, const rubick_plan *h_plans, int P, const rubick_grid *h_grid)
{
    CHECK_CTX(ctx);
    if (!h_plans || P <= 0) return fail(ctx, RUBICK_EINVAL, "plans: need a positive multiple of 4");
    std::vector<NormPlan> np_list((size_t(P)));
    for (int i = 0; i < P; ++i) {
        const rubick_plan &pl = h_plans[i];
        if (pl.log2d > 15 || pl.log2t > 15 || pl.log2p > 15) return fail(ctx, RUBICK_EINVAL, "plans: field out of range");
        np_list[i] = NormPlan{1 << pl.log2d, 1 << pl.log2t, 1 << pl.log2p, pl.zero, pl.gc, pl.off, pl.g_level, pl.disabled, 0};
    }
    return install_space(ctx, np_list.data(), P, h_grid, false);
}

int rubick_set_space_wide(rubick_ctx *ctx, const rubick_plan_wide *h_plans, int P, const rubick_grid *h_grid)
{
    CHECK_CTX(ctx);
    if (!h_plans || P <= 0) return fail(ctx, RUBICK_EINVAL, "plans: need a positive multiple of 4");
    std::vector<NormPlan> np_list((size_t(P)));
    for (int i = 0; i < P; ++i) {
        const rubick_plan_wide &pl = h_plans[i];
        np_list[i] = NormPlan{pl.d, pl.t, pl.p, pl.zero, pl.gc, pl.off, pl.g_level, pl.disabled, pl.accum};
    }
    return install_space(ctx, np_list.data(), P, h_grid, true);
}

int rubick_set_placement(rubick_ctx *ctx, int align)
{
    CHECK_CTX(ctx);
    if (!ctx->has_space) return fail(ctx, RUBICK_ESTATE, "no plan space: call rubick_set_space first");
    if (align < 0 || align >= ctx->space.Gn || (align & (align - 1))) return fail(ctx, RUBICK_EINVAL, "placement: align must be 0 or a power of two below gpus_per_node");
    std::vector<QuadDesc> quads;
    std::vector<WideQuad> wquads;
    build_quads(ctx->norm_plans, ctx->space.g_levels, ctx->space.Gn, ctx->space.wide != 0, align, quads, wquads);
    int rc = upload_quads(ctx, quads, wquads);
    if (rc) return rc;
    ctx->placement_align = align;
    ctx->inc_J = 0;                     // cached tables of the incremental events belong to the other class
    return RUBICK_OK;
}

int rubick_enumerate_plans_wide(const int32_t *h_g_levels, int nG, int n_accum, rubick_plan_wide *h_out, int cap,
                                int *n_out, int32_t *h_group_off)
{
    if (!h_g_levels || nG < 1 || nG > RUBICK_MAX_G_LEVELS || !n_out || cap < 0 || (cap > 0 && !h_out)) return RUBICK_EINVAL;
    if (n_accum < 1 || n_accum > 8) return RUBICK_EINVAL;
    for (int i = 0; i < nG; ++i)
        if (h_g_levels[i] <= 0 || h_g_levels[i] > 32768 || (i && h_g_levels[i] <= h_g_levels[i - 1])) return RUBICK_EINVAL;
    int n = 0;
    for (int gi = 0; gi < nG; ++gi) {
        if (h_group_off) h_group_off[gi] = n;
        const int g = h_g_levels[gi];
        for (int t = 1; t <= g; ++t) {
            if (g % t) continue;
            for (int p = 1; p <= g / t; ++p) {
                if ((g / t) % p) continue;
                for (int ga = 0; ga < n_accum; ++ga)
                    for (int z = 0; z < 4; ++z)
                        for (int v = 0; v < 4; ++v, ++n)
                            if (n < cap) {
                                rubick_plan_wide &pl = h_out[n];
                                pl.d = uint16_t(g / (t * p)); pl.t = uint16_t(t); pl.p = uint16_t(p);
                                pl.zero = uint8_t(z); pl.gc = uint8_t(v >> 1); pl.off = uint8_t(v & 1);
                                pl.g_level = uint8_t(gi); pl.disabled = 0; pl.accum = uint8_t(ga);
                            }
            }
        }
    }
    if (h_group_off) h_group_off[nG] = n;
    *n_out = n;
    return RUBICK_OK;
}

static int check_ready(rubick_ctx *ctx, int J)
{
    if (!ctx->has_space) return fail(ctx, RUBICK_ESTATE, "no plan space: call rubick_set_space first");
    if (J < 0) return fail(ctx, RUBICK_EINVAL, "negative job count");
    if (cudaSetDevice(ctx->device) != cudaSuccess) return fail(ctx, RUBICK_ECUDA, "cudaSetDevice failed");
    return RUBICK_OK;
}

int rubick_eval_candidates(rubick_ctx *ctx, const rubick_job *d_jobs, int J, float *d_thr, uint32_t *d_feas)
{
    CHECK_CTX(ctx);
    int rc = check_ready(ctx, J);
    if (rc) return rc;
    if (J == 0) return RUBICK_OK;
    if (!d_jobs || !d_thr || !d_feas) return fail(ctx, RUBICK_EINVAL, "null pointer");
    if ((reinterpret_cast<uintptr_t>(d_thr) & 15) || (reinterpret_cast<uintptr_t>(d_feas) & 15) || (reinterpret_cast<uintptr_t>(d_jobs) & 15))
        return fail(ctx, RUBICK_EINVAL, "d_jobs, d_thr and d_feas must be 16-byte aligned");
    if (int64_t(J) * ctx->space.Q >= (int64_t(1) << 31)) return fail(ctx, RUBICK_EINVAL, "J * P / 4 must stay below 2^31: evaluate in job tiles");
    CUDA_TRY(ctx, launch_eval(ctx->space, ctx->d_quads, ctx->d_wide_quads, d_jobs, J, d_thr, d_feas, ctx->stream), "launch eval_candidates");
    return RUBICK_OK;
}

int rubick_best_plan(rubick_ctx *ctx, const float *d_thr, const uint32_t *d_feas, int J, unsigned flags,
                     float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g)
{
    CHECK_CTX(ctx);
    int rc = check_ready(ctx, J);
    if (rc) return rc;
    if (J == 0) return RUBICK_OK;
    if (!d_thr || !d_feas || !d_best_val || !d_best_plan || !d_best_g) return fail(ctx, RUBICK_EINVAL, "null pointer");
    if ((reinterpret_cast<uintptr_t>(d_thr) & 15) || (reinterpret_cast<uintptr_t>(d_feas) & 15))
        return fail(ctx, RUBICK_EINVAL, "d_thr and d_feas must be 16-byte aligned");
    if (flags & ~RUBICK_BEST_RAW) return fail(ctx, RUBICK_EINVAL, "unknown flag");
    if ((rc = ensure(ctx, ctx->d_best_todo, ctx->cap_best_todo, size_t(J) + 1))) return rc;
    CUDA_TRY(ctx, launch_best(ctx->space, d_thr, d_feas, J, flags, d_best_val, d_best_plan, d_best_g, ctx->d_status,
                              ctx->d_best_todo, ctx->num_sms, ctx->stream),
             "launch best_plan");
    return RUBICK_OK;
}

int rubick_curves(rubick_ctx *ctx, const rubick_job *d_jobs, int J, unsigned flags, uint32_t *d_feas,
                  float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g)
{
    CHECK_CTX(ctx);
    int rc = check_ready(ctx, J);
    if (rc) return rc;
    if (J == 0) return RUBICK_OK;
    if (!d_jobs || !d_feas || !d_best_val || !d_best_plan || !d_best_g) return fail(ctx, RUBICK_EINVAL, "null pointer");
    if ((reinterpret_cast<uintptr_t>(d_feas) & 15) || (reinterpret_cast<uintptr_t>(d_jobs) & 15))
        return fail(ctx, RUBICK_EINVAL, "d_jobs and d_feas must be 16-byte aligned");
    if (flags & ~RUBICK_BEST_RAW) return fail(ctx, RUBICK_EINVAL, "unknown flag");
    CUDA_TRY(ctx, launch_curves(ctx->space, ctx->d_quads, ctx->d_wide_quads, d_jobs, J, flags, d_feas, d_best_val, d_best_plan, d_best_g, ctx->stream),
             "launch curves");
    return RUBICK_OK;
}

int rubick_marginal_gain(rubick_ctx *ctx, const rubick_job *d_jobs, int J, const float *d_curve_val,
                         const rubick_assignment *d_state,
                         float *d_gain_gpu, float *d_gain_cpu, int32_t *d_next_g, int32_t *d_next_c)
{
    CHECK_CTX(ctx);
    int rc = check_ready(ctx, J);
    if (rc) return rc;
    if (J == 0) return RUBICK_OK;
    if (!d_jobs || !d_curve_val || !d_state || !d_gain_gpu || !d_gain_cpu || !d_next_g || !d_next_c) return fail(ctx, RUBICK_EINVAL, "null pointer");
    CUDA_TRY(ctx, launch_gain(ctx->space, d_jobs, J, d_curve_val, d_state, d_gain_gpu, d_gain_cpu, d_next_g, d_next_c, ctx->stream),
             "launch marginal_gain");
    return RUBICK_OK;
}

int rubick_min_resources(rubick_ctx *ctx, const float *d_thr, const uint32_t *d_feas, const float *d_curve_val, int J,
                         const rubick_request *d_req, int32_t *d_gmin_idx, int32_t *d_cmin_idx, float *d_baseline)
{
    CHECK_CTX(ctx);
    int rc = check_ready(ctx, J);
    if (rc) return rc;
    if (J == 0) return RUBICK_OK;
    if (!d_thr || !d_feas || !d_curve_val || !d_req || !d_gmin_idx || !d_cmin_idx || !d_baseline) return fail(ctx, RUBICK_EINVAL, "null pointer");
    CUDA_TRY(ctx, launch_min_resources(ctx->space, ctx->d_quads, d_thr, d_feas, d_curve_val, J, d_req, d_gmin_idx, d_cmin_idx,
                                       d_baseline, ctx->stream),
             "launch min_resources");
    return RUBICK_OK;
}

int rubick_fit_models(rubick_ctx *ctx, const rubick_job *d_jobs, int J, const rubick_sample *d_samples, int S,
                      int sweeps, double *d_theta, double *d_rmsle)
{
    CHECK_CTX(ctx);
    int rc = check_ready(ctx, J);
    if (rc) return rc;
    if (J == 0) return RUBICK_OK;
    if (!d_jobs || !d_samples || !d_theta || !d_rmsle) return fail(ctx, RUBICK_EINVAL, "null pointer");
    if (S < 1 || S > 4096) return fail(ctx, RUBICK_EINVAL, "1 .. 4096 sample slots per model");
    if (sweeps < 0 || sweeps > 64) return fail(ctx, RUBICK_EINVAL, "0 .. 64 sweeps");
    if ((reinterpret_cast<uintptr_t>(d_samples) & 7) || (reinterpret_cast<uintptr_t>(d_theta) & 7) || (reinterpret_cast<uintptr_t>(d_rmsle) & 7))
        return fail(ctx, RUBICK_EINVAL, "d_samples, d_theta and d_rmsle must be 8-byte aligned");
    CUDA_TRY(ctx, launch_fit(ctx->env, ctx->d_quads, ctx->space.wide ? ctx->d_wide_quads : nullptr, ctx->space.P, d_jobs, J, d_samples, S, sweeps, d_theta, d_rmsle, ctx->stream),
             "launch fit_models");
    return RUBICK_OK;
}

// enqueue the round and leave the step count in ctx->d_steps
static int enqueue_round(rubick_ctx *ctx, const rubick_job *d_jobs, int J, const float *d_cv, const int32_t *d_cp,
                         const int32_t *d_cg, const uint32_t *d_feas, const rubick_cluster *cl, int max_steps,
                         rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log, const int4 *d_top = nullptr)
{
    const int N = cl->n_nodes, T = cl->n_tenants;
    if (T > 0) {
        // interleave (GPUs, cores) per tenant; the staging vector lives in the context until the next round
        cudaStreamSynchronize(ctx->stream);
        ctx->h_quota.resize(size_t(2) * T);
        for (int t = 0; t < T; ++t) { ctx->h_quota[2 * t] = cl->quota_gpus[t]; ctx->h_quota[2 * t + 1] = cl->quota_cpus[t]; }
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_quota, ctx->h_quota.data(), size_t(8) * T, cudaMemcpyHostToDevice, ctx->stream), "upload quotas");
    }
    const bool fast = round_fast_supported(ctx->space, J, N);
    const size_t need = fast ? round_fast_scratch_need(ctx->space, J, N) : round_scratch_need(ctx->space, J, N);
    if (need > ctx->round_scratch_bytes) {
        if (ctx->d_round_scratch) { cudaStreamSynchronize(ctx->stream); cudaFree(ctx->d_round_scratch); ctx->d_round_scratch = nullptr; ctx->round_scratch_bytes = 0; }
        CUDA_TRY(ctx, cudaMalloc(&ctx->d_round_scratch, need), "cudaMalloc (round scratch)");
        ctx->round_scratch_bytes = need;
    }
    if (fast)
        CUDA_TRY(ctx, launch_round_fast(ctx->space, d_jobs, J, d_cv, d_cp, d_cg, d_feas, N, max_steps, d_out, d_node_out, d_step_log,
                                        ctx->d_round_scratch, ctx->d_quota, T, ctx->d_status, ctx->d_steps, ctx->stream, d_top),
                 "launch greedy_round (fast path)");
    else
        CUDA_TRY(ctx, launch_round(ctx->space, d_jobs, J, d_cv, d_cp, d_cg, d_feas, N, max_steps, d_out, d_node_out, d_step_log,
                                   ctx->d_round_scratch, ctx->d_quota, T, ctx->d_status, ctx->d_steps, ctx->stream),
                 "launch greedy_round");
    return RUBICK_OK;
}

// wait for the round, fetch the step count and the cap flag
static int finish_round(rubick_ctx *ctx, int32_t *h_steps)
{
    uint32_t two[2] = {0, 0};
    CUDA_TRY(ctx, cudaMemcpyAsync(two, ctx->d_status, 8, cudaMemcpyDeviceToHost, ctx->stream), "read round status");
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
    if (h_steps) *h_steps = int32_t(two[1]);
    if (two[0] & DS_STEP_CAP) {
        const uint32_t cleared = two[0] & ~DS_STEP_CAP;
        cudaMemcpyAsync(ctx->d_status, &cleared, 4, cudaMemcpyHostToDevice, ctx->stream);
        cudaStreamSynchronize(ctx->stream);
        return fail(ctx, RUBICK_ESTEPS, "greedy round stopped at max_steps");
    }
    if (two[0] & DS_FEAS_NOT_THRESHOLD) {
        cudaMemset(ctx->d_status, 0, 4);
        return fail(ctx, RUBICK_ESTATE, "a feasibility word is not a threshold in the memory-level index");
    }
    if (two[0] & DS_BAD_PREV) {
        cudaMemset(ctx->d_status, 0, 4);
        return fail(ctx, RUBICK_ESTATE, "incremental round: the previous allocation does not fit the grid or the cluster");
    }
    return RUBICK_OK;
}

static int check_round_args(rubick_ctx *ctx, int J, const rubick_cluster *h_cluster, int max_steps)
{
    int rc = check_ready(ctx, J);
    if (rc) return rc;
    if (!h_cluster || h_cluster->n_nodes < 1 || h_cluster->n_nodes > RUBICK_MAX_NODES) return fail(ctx, RUBICK_EINVAL, "cluster: 1 .. RUBICK_MAX_NODES nodes");
    if (h_cluster->n_tenants < 0 || h_cluster->n_tenants > RUBICK_MAX_TENANTS || (h_cluster->n_tenants > 0 && (!h_cluster->quota_gpus || !h_cluster->quota_cpus)))
        return fail(ctx, RUBICK_EINVAL, "cluster: 0 .. RUBICK_MAX_TENANTS tenants with both quota arrays");
    if (max_steps < 0) return fail(ctx, RUBICK_EINVAL, "negative max_steps");
    if (J >= (1 << 29)) return fail(ctx, RUBICK_EINVAL, "too many jobs");
    return RUBICK_OK;
}

int rubick_greedy_round(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                        const float *d_curve_val, const int32_t *d_curve_plan, const int32_t *d_curve_g,
                        const uint32_t *d_feas, const rubick_cluster *h_cluster, int max_steps,
                        rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                        int32_t *h_steps)
{
    CHECK_CTX(ctx);
    int rc = check_round_args(ctx, J, h_cluster, max_steps);
    if (rc) return rc;
    if (J > 0 && (!d_jobs || !d_curve_val || !d_curve_plan || !d_curve_g || !d_feas || !d_out)) return fail(ctx, RUBICK_EINVAL, "null pointer");
    rc = enqueue_round(ctx, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas, h_cluster, max_steps, d_out,
                       d_node_out, d_step_log);
    if (rc) return rc;
    return finish_round(ctx, h_steps);
}

int rubick_incremental_round(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                             const float *d_curve_val, const int32_t *d_curve_plan, const int32_t *d_curve_g,
                             const uint32_t *d_feas, const rubick_cluster *h_cluster,
                             const rubick_assignment *d_prev, const rubick_node *d_prev_nodes,
                             const rubick_reconf *d_reconf, float theta, int max_steps,
                             rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                             int32_t *h_steps)
{
    CHECK_CTX(ctx);
    int rc = check_round_args(ctx, J, h_cluster, max_steps);
    if (rc) return rc;
    if (J > 0 && (!d_jobs || !d_curve_val || !d_curve_plan || !d_curve_g || !d_feas || !d_out)) return fail(ctx, RUBICK_EINVAL, "null pointer");
    if ((d_prev == nullptr) != (d_prev_nodes == nullptr)) return fail(ctx, RUBICK_EINVAL, "d_prev and d_prev_nodes come together");
    if (ctx->space.Gn > 32) return fail(ctx, RUBICK_EINVAL, "incremental round: at most 32 GPUs per node");
    if (!(theta == theta)) return fail(ctx, RUBICK_EINVAL, "theta is not a number");
    const int N = h_cluster->n_nodes, T = h_cluster->n_tenants;
    if (T > 0) {
        cudaStreamSynchronize(ctx->stream);
        ctx->h_quota.resize(size_t(2) * T);
        for (int t = 0; t < T; ++t) { ctx->h_quota[2 * t] = h_cluster->quota_gpus[t]; ctx->h_quota[2 * t + 1] = h_cluster->quota_cpus[t]; }
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_quota, ctx->h_quota.data(), size_t(8) * T, cudaMemcpyHostToDevice, ctx->stream), "upload quotas");
    }
    const size_t need = incr_scratch_need(ctx->space, J, N);
    if (need > ctx->round_scratch_bytes) {
        if (ctx->d_round_scratch) { cudaStreamSynchronize(ctx->stream); cudaFree(ctx->d_round_scratch); ctx->d_round_scratch = nullptr; ctx->round_scratch_bytes = 0; }
        CUDA_TRY(ctx, cudaMalloc(&ctx->d_round_scratch, need), "cudaMalloc (round scratch)");
        ctx->round_scratch_bytes = need;
    }
    CUDA_TRY(ctx, launch_round_incremental(ctx->space, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas, N, max_steps,
                                           d_prev, d_prev_nodes, d_reconf, theta, d_out, d_node_out, d_step_log,
                                           ctx->d_round_scratch, ctx->d_quota, T, ctx->d_status, ctx->d_steps, ctx->stream),
             "launch incremental_round");
    return finish_round(ctx, h_steps);
}

// mask and curves for d_jobs[0..J) into context scratch
static int enqueue_tables(rubick_ctx *ctx, const rubick_job *d_jobs, int J)
{
    const Space &sp = ctx->space;
    ctx->inc_J = 0;                     // the table scratch is about to be rewritten
    int rc;
    if ((rc = ensure(ctx, ctx->d_feas, ctx->cap_feas, size_t(J) * sp.P))) return rc;
    const size_t curve = size_t(J) * sp.nG * sp.nC * sp.nM;
    if (curve > ctx->cap_curve) {
        // the three tables grow together; if one allocation fails none of them is kept, so that no later call
        // (whose smaller J would skip this branch) can hand a freed or null table to a kernel
        size_t c1 = ctx->cap_curve, c2 = ctx->cap_curve, c3 = ctx->cap_curve;
        ctx->cap_curve = 0;
        if ((rc = ensure(ctx, ctx->d_cv, c1, curve)) || (rc = ensure(ctx, ctx->d_cp, c2, curve)) || (rc = ensure(ctx, ctx->d_cg, c3, curve))) {
            cudaFree(ctx->d_cv); cudaFree(ctx->d_cp); cudaFree(ctx->d_cg);
            ctx->d_cv = nullptr; ctx->d_cp = nullptr; ctx->d_cg = nullptr;
            return rc;
        }
        ctx->cap_curve = curve;
    }
    if ((rc = ensure(ctx, ctx->d_top, ctx->cap_top, size_t(J) * sp.nG * sp.nC))) return rc;
    // a round only needs the curves: the one-pass kernel never writes the candidate table; it leaves the top memory level
    // once more in packed form for the round's preparation
    CUDA_TRY(ctx, launch_curves(sp, ctx->d_quads, ctx->d_wide_quads, d_jobs, J, 0u, ctx->d_feas, ctx->d_cv, ctx->d_cp, ctx->d_cg, ctx->stream, ctx->d_top),
             "launch curves");
    return RUBICK_OK;
}

int rubick_schedule_round(rubick_ctx *ctx, const rubick_job *d_jobs, int J, const rubick_cluster *h_cluster,
                          int max_steps, rubick_assignment *d_out, rubick_node *d_node_out, int32_t *h_steps)
{
    CHECK_CTX(ctx);
    int rc = check_round_args(ctx, J, h_cluster, max_steps);
    if (rc) return rc;
    if (J > 0 && (!d_jobs || !d_out)) return fail(ctx, RUBICK_EINVAL, "null pointer");
    if (J > 0 && (reinterpret_cast<uintptr_t>(d_jobs) & 15)) return fail(ctx, RUBICK_EINVAL, "d_jobs must be 16-byte aligned");
    if ((rc = enqueue_tables(ctx, d_jobs, J))) return rc;
    if ((rc = enqueue_round(ctx, d_jobs, J, ctx->d_cv, ctx->d_cp, ctx->d_cg, ctx->d_feas, h_cluster, max_steps, d_out, d_node_out, nullptr, ctx->d_top))) return rc;
    return finish_round(ctx, h_steps);
}

int rubick_schedule_round_host(rubick_ctx *ctx, const rubick_job *h_jobs, int J, const rubick_cluster *h_cluster,
                               int max_steps, rubick_assignment *h_out, rubick_node *h_node_out, int32_t *h_steps)
{
    CHECK_CTX(ctx);
    int rc = check_round_args(ctx, J, h_cluster, max_steps);
    if (rc) return rc;
    if (J > 0 && (!h_jobs || !h_out)) return fail(ctx, RUBICK_EINVAL, "null pointer");
    const int N = h_cluster->n_nodes;
    if ((rc = ensure(ctx, ctx->d_jobs_stage, ctx->cap_jobs, size_t(J > 0 ? J : 1)))) return rc;
    if ((rc = ensure(ctx, ctx->d_out_stage, ctx->cap_out, size_t(J > 0 ? J : 1)))) return rc;
    if ((rc = ensure(ctx, ctx->d_node_stage, ctx->cap_node, size_t(N)))) return rc;
    if (J > 0) CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_jobs_stage, h_jobs, size_t(J) * sizeof(rubick_job), cudaMemcpyHostToDevice, ctx->stream), "copy jobs to device");
    if ((rc = enqueue_tables(ctx, ctx->d_jobs_stage, J))) return rc;
    if ((rc = enqueue_round(ctx, ctx->d_jobs_stage, J, ctx->d_cv, ctx->d_cp, ctx->d_cg, ctx->d_feas, h_cluster, max_steps, ctx->d_out_stage,
                            ctx->d_node_stage, nullptr, ctx->d_top))) return rc;
    if (J > 0) CUDA_TRY(ctx, cudaMemcpyAsync(h_out, ctx->d_out_stage, size_t(J) * sizeof(rubick_assignment), cudaMemcpyDeviceToHost, ctx->stream), "copy assignments to host");
    if (h_node_out) CUDA_TRY(ctx, cudaMemcpyAsync(h_node_out, ctx->d_node_stage, size_t(N) * sizeof(rubick_node), cudaMemcpyDeviceToHost, ctx->stream), "copy node states to host");
    return finish_round(ctx, h_steps);
}

// tables of the listed slots only (the others keep what an earlier call computed)
static int enqueue_tables_of(rubick_ctx *ctx, const rubick_job *d_jobs, const int32_t *h_slots, int n)
{
    const Space &sp = ctx->space;
    const size_t per_job = size_t(sp.nG) * sp.nC * sp.nM;
    for (int i = 0; i < n;) {
        int run = 1;                    // consecutive slots go through the kernel together
        while (i + run < n && h_slots[i + run] == h_slots[i] + run) ++run;
        const int s0 = h_slots[i];
        CUDA_TRY(ctx, launch_curves(sp, ctx->d_quads, ctx->d_wide_quads, d_jobs + s0, run, 0u, ctx->d_feas + size_t(s0) * sp.P, ctx->d_cv + s0 * per_job,
                                    ctx->d_cp + s0 * per_job, ctx->d_cg + s0 * per_job, ctx->stream),
                 "launch curves");
        i += run;
    }
    return RUBICK_OK;
}

int rubick_incremental_event_host(rubick_ctx *ctx, const rubick_job *h_jobs, int J, const rubick_cluster *h_cluster,
                                  const int32_t *h_changed, int n_changed, const rubick_reconf *h_reconf, float theta,
                                  int restart, int max_steps, rubick_assignment *h_out, rubick_node *h_node_out,
                                  int32_t *h_steps)
{
    CHECK_CTX(ctx);
    int rc = check_round_args(ctx, J, h_cluster, max_steps);
    if (rc) return rc;
    if (J < 1 || !h_jobs || !h_out) return fail(ctx, RUBICK_EINVAL, "null pointer or no job slots");
    if (n_changed > 0 && !h_changed) return fail(ctx, RUBICK_EINVAL, "n_changed > 0 without the slot list");
    if (ctx->space.Gn > 32) return fail(ctx, RUBICK_EINVAL, "incremental round: at most 32 GPUs per node");
    if (!(theta == theta)) return fail(ctx, RUBICK_EINVAL, "theta is not a number");
    const int N = h_cluster->n_nodes, T = h_cluster->n_tenants;
    const bool fresh = restart || ctx->inc_J != J || ctx->inc_N != N;
    if (!fresh)
        for (int i = 0; i < n_changed; ++i)
            if (h_changed[i] < 0 || h_changed[i] >= J) return fail(ctx, RUBICK_EINVAL, "changed slot out of range");
    for (int i = 0; i < 2; ++i) {
        if ((rc = ensure(ctx, ctx->d_inc_state[i], ctx->cap_inc_state[i], size_t(J)))) return rc;
        if ((rc = ensure(ctx, ctx->d_inc_nodes[i], ctx->cap_inc_nodes[i], size_t(N)))) return rc;
    }
    if ((rc = ensure(ctx, ctx->d_inc_jobs, ctx->cap_inc_jobs, size_t(J)))) return rc;
    if ((rc = ensure(ctx, ctx->d_inc_reconf, ctx->cap_inc_reconf, size_t(J)))) return rc;
    const bool all = fresh || n_changed < 0;
    if (all) {
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_inc_jobs, h_jobs, size_t(J) * sizeof(rubick_job), cudaMemcpyHostToDevice, ctx->stream), "copy jobs to device");
        if ((rc = enqueue_tables(ctx, ctx->d_inc_jobs, J))) return rc;
    } else {
        for (int i = 0; i < n_changed; ++i)
            CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_inc_jobs + h_changed[i], h_jobs + h_changed[i], sizeof(rubick_job), cudaMemcpyHostToDevice, ctx->stream), "copy a job to device");
        if ((rc = enqueue_tables_of(ctx, ctx->d_inc_jobs, h_changed, n_changed))) return rc;
    }
    if (h_reconf) CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_inc_reconf, h_reconf, size_t(J) * sizeof(rubick_reconf), cudaMemcpyHostToDevice, ctx->stream), "copy gate inputs to device");
    if (T > 0) {
        cudaStreamSynchronize(ctx->stream);
        ctx->h_quota.resize(size_t(2) * T);
        for (int t = 0; t < T; ++t) { ctx->h_quota[2 * t] = h_cluster->quota_gpus[t]; ctx->h_quota[2 * t + 1] = h_cluster->quota_cpus[t]; }
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_quota, ctx->h_quota.data(), size_t(8) * T, cudaMemcpyHostToDevice, ctx->stream), "upload quotas");
    }
    const size_t need = incr_scratch_need(ctx->space, J, N);
    if (need > ctx->round_scratch_bytes) {
        if (ctx->d_round_scratch) { cudaStreamSynchronize(ctx->stream); cudaFree(ctx->d_round_scratch); ctx->d_round_scratch = nullptr; ctx->round_scratch_bytes = 0; }
        CUDA_TRY(ctx, cudaMalloc(&ctx->d_round_scratch, need), "cudaMalloc (round scratch)");
        ctx->round_scratch_bytes = need;
    }
    const int cur = ctx->inc_cur, nxt = 1 - cur;
    CUDA_TRY(ctx, launch_round_incremental(ctx->space, ctx->d_inc_jobs, J, ctx->d_cv, ctx->d_cp, ctx->d_cg, ctx->d_feas, N, max_steps,
                                           fresh ? nullptr : ctx->d_inc_state[cur], fresh ? nullptr : ctx->d_inc_nodes[cur],
                                           h_reconf ? ctx->d_inc_reconf : nullptr, theta, ctx->d_inc_state[nxt], ctx->d_inc_nodes[nxt],
                                           nullptr, ctx->d_round_scratch, ctx->d_quota, T, ctx->d_status, ctx->d_steps, ctx->stream),
             "launch incremental_round");
    // the status first: a round that was refused has written no result, and the caller's buffers stay as they are
    rc = finish_round(ctx, h_steps);
    if (rc != RUBICK_OK && rc != RUBICK_ESTEPS) { ctx->inc_J = 0; return rc; }
    ctx->inc_cur = nxt; ctx->inc_J = J; ctx->inc_N = N;
    CUDA_TRY(ctx, cudaMemcpyAsync(h_out, ctx->d_inc_state[nxt], size_t(J) * sizeof(rubick_assignment), cudaMemcpyDeviceToHost, ctx->stream), "copy assignments to host");
    if (h_node_out) CUDA_TRY(ctx, cudaMemcpyAsync(h_node_out, ctx->d_inc_nodes[nxt], size_t(N) * sizeof(rubick_node), cudaMemcpyDeviceToHost, ctx->stream), "copy node states to host");
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
    return rc;
}

}  // extern "C"
