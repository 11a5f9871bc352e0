// Incremental scheduling round (paper Section 5.2: Algorithm 1 with its shrink step, started from
// the previous allocation, and "Incorporating reconfiguration penalty").
//
// What is decided, in the order it is decided:
//   * job slots keep their index between rounds; a running job carries its GPUs, cores, memory, plan
//     and node(s) over;
//   * gate: a running job may be touched only if T > 0 and (T - (N + 1) * delta) / T > theta; the
//     others are pinned for the round;
//   * a running, unpinned single-node job offers shrink steps: GPUs down to the next lower level whose
//     own plans run (not below its guaranteed minimum; a best-effort job without such a level is
//     preempted), cores down one level; the slope of a step is the weighted value lost per unit;
//   * an increment that does not fit free resources may take from the lowest-slope offers on its node
//     while its own gain per unit is larger (unconditionally for a queued guaranteed job placed at
//     its minimum); the attempt is all or nothing; shrunk jobs do not grow again in the round;
//   * Phase A places queued guaranteed jobs at their minimum (free resources first, else exchange on
//     the first node where it works) within their tenant's remaining quota; Phase B takes the
//     largest gain that fits free resources, and only when nothing fits, the largest gain by exchange.
// All comparisons are single precision with one rounding per operation, as in the grow-only round.
//
// One persistent CTA, like the plain round: per step every warp rebuilds the first-fit table, every
// thread scans its jobs for the best increment that fits and the best increment at all, a block-wide
// argmax picks the winner and warp 0 commits.  An exchange is worked out by warp 0 alone: every node
// keeps the list of its single-node jobs (at most gpus_per_node of them, since each holds a GPU), so
// lane i owns the i-th job of the node, works out what that job would give up and at what slope, and
// a warp argmin picks the victim of each step.  All changes of an attempt live in registers until
// the increment itself has been committed; a failed attempt leaves no trace.

#include "round_plain.cuh"

namespace rubick {

constexpr int MAX_EXCHANGE_STEPS = 64;      // shrink steps one exchange may take

// roles of a job in this round: [5:0] minimum g level + 1 (0 = none) | [12:6] minimum c level |
// [13] guaranteed | [14] pinned by the gate | [15] slot in use | [16] shrunk in this round
__device__ __forceinline__ int rl_min_gi(uint32_t r) { return int(r & 63u) - 1; }
__device__ __forceinline__ int rl_min_ci(uint32_t r) { return int((r >> 6) & 127u); }
__device__ __forceinline__ bool rl_guaranteed(uint32_t r) { return (r >> 13) & 1u; }
__device__ __forceinline__ bool rl_pinned(uint32_t r) { return (r >> 14) & 1u; }
__device__ __forceinline__ bool rl_active(uint32_t r) { return (r >> 15) & 1u; }

struct JobRegs { HotA a; HotB b; };

struct NodeFree { int g, c; int64_t m; };

// what a running single-node job would give up next
struct Offer { bool ok; int gi2, ci2; float slope; };

__device__ Offer shrink_offer(const Space &sp, const float *__restrict__ cv, const int32_t *__restrict__ cp,
                              const int32_t *__restrict__ cg, int v, const JobRegs &s, uint32_t roles, int type)
{
    Offer o; o.ok = false; o.gi2 = -1; o.ci2 = pk_ci(s.a.packed); o.slope = 0.0f;
    const int gi = pk_gi(s.a.packed), ci = pk_ci(s.a.packed);
    if (gi < 0 || sp.g_levels[gi] > sp.Gn) return o;
    const int mt = sp.nM - 1;
    const float w = s.b.w;
    const float vcur = __fmul_rn(w, s.b.val);
    const bool guaranteed = rl_guaranteed(roles);
    if (type == 0) {
        if (guaranteed && rl_min_gi(roles) < 0) return o;
        const int lo = guaranteed ? rl_min_gi(roles) : 0;
        for (int i = gi - 1; i >= lo; --i) {
            const size_t x = curve_idx(sp, v, i, ci, mt);
            if (cp[x] >= 0 && cg[x] == sp.g_levels[i]) {
                o.ok = true; o.gi2 = i;
                o.slope = __fdiv_rn(__fsub_rn(vcur, __fmul_rn(w, cv[x])), float(sp.g_levels[gi] - sp.g_levels[i]));
                return o;
            }
        }
        if (guaranteed) return o;
        o.ok = true; o.gi2 = -1;                    // preemption
        o.slope = __fdiv_rn(__fsub_rn(vcur, __fmul_rn(w, 0.0f)), float(sp.g_levels[gi]));
        return o;
    }
    const int lo = guaranteed ? rl_min_ci(roles) : 0;
    if (ci - 1 < lo) return o;
    const size_t x = curve_idx(sp, v, gi, ci - 1, mt);
    if (cp[x] < 0 || cg[x] != sp.g_levels[gi]) return o;
    o.ok = true; o.gi2 = gi; o.ci2 = ci - 1;
    o.slope = __fdiv_rn(__fsub_rn(vcur, __fmul_rn(w, cv[x])), float(sp.c_levels[ci] - sp.c_levels[ci - 1]));
    return o;
}

// Job j (state s, on `node` already when `stay`) takes (gi2, ci2) on that node, whose free amounts are
// nf: host-memory level that fits, curve look-up there (GetBestPlan), memory of that plan (AllocMem).
// Returns false and changes nothing when it does not fit.  One thread.
__device__ bool take_on_node(const Space &sp, const float *__restrict__ cv, const int32_t *__restrict__ cp,
                             const int32_t *__restrict__ cg, const uint32_t *__restrict__ feas, int j, JobRegs &s,
                             NodeFree &nf, int node, bool stay, int gi2, int ci2, bool need_gain)
{
    const int gi = pk_gi(s.a.packed), ci = pk_ci(s.a.packed);
    const bool alloc = gi >= 0;
    const int g = alloc ? sp.g_levels[gi] : 0, c = alloc ? sp.c_levels[ci] : 0;
    const int64_t m_cur = alloc ? sp.m_levels[s.b.f_level] : 0;
    const int g2 = sp.g_levels[gi2], c2 = sp.c_levels[ci2];
    const int64_t avail = nf.m + ((stay && alloc) ? m_cur : 0);
    int mi = -1;
    for (int i = 0; i < sp.nM; ++i) if (sp.m_levels[i] <= avail) mi = i;
    if (mi < 0) return false;
    const size_t o = curve_idx(sp, j, gi2, ci2, mi);
    const float v = cv[o];
    const int plan = cp[o], gu = cg[o];
    if (plan < 0 || plan >= sp.P || !(v > 0.0f) || gu != g2) return false;
    if (need_gain && alloc && !(v > s.b.val)) return false;
    const uint32_t word = feas[size_t(j) * sp.P + plan];
    const int f = __ffs(word) - 1;
    if (f < 0 || f > mi) return false;
    if (stay && alloc) { nf.g += g; nf.c += c; nf.m += m_cur; }
    nf.g -= g2; nf.c -= c2; nf.m -= sp.m_levels[f];
    s.a.node = node;
    s.a.packed = pack(gi2, ci2, -1, false, pk_fz_g(s.a.packed), pk_fz_c(s.a.packed));
    s.b.val = v; s.b.plan = plan; s.b.f_level = f;
    return true;
}

struct IncrShared {
    unsigned long long red[4][ROUND_WARPS];
    float redf[2][ROUND_WARPS];
    int redi[3][ROUND_WARPS];
    int n_empty;
    int sel_j, which;         // the step's job and kind: 0 / 1 GPU / CPU increment on free resources, 2 / 3 by exchange
    int steps, capped;
    int changed;              // the last step changed the cluster: the first-fit table is stale
    int batch;                // this iteration sorts out hopeless exchange candidates in bulk
    int most_c[33];           // most free cores among the nodes with at least g free GPUs (g <= 32)
    float min_slope[2];       // lowest offered slope over all nodes, GPUs / cores
    int max_free[2];          // most free GPUs / cores on any node
};

struct NodeLists {            // single-node jobs of every node
    int32_t *cnt;             // [N] shared memory
    int32_t *jobs;            // [N][Gn] global scratch
    int Gn;
};

__device__ __forceinline__ void list_add(NodeLists &nl, int n, int j) { nl.jobs[size_t(n) * nl.Gn + nl.cnt[n]] = j; nl.cnt[n] += 1; }
__device__ __forceinline__ void list_remove(NodeLists &nl, int n, int j)
{
    int32_t *l = nl.jobs + size_t(n) * nl.Gn;
    const int c = nl.cnt[n];
    for (int i = 0; i < c; ++i)
        if (l[i] == j) { l[i] = l[c - 1]; nl.cnt[n] = c - 1; return; }
}

// An exchange for a queued job can only work on a node whose free amounts plus everything its unpinned
// single-node jobs hold cover the job: a cheap test that spares hopeless attempts.  Lane i looks at node
// base + i; returns the ballot of the nodes that pass.
__device__ unsigned nodes_could_serve(const Space &sp, const Cluster &cl, const NodeLists &nl, const HotA *hotA,
                                      const uint32_t *roles, int base, int g2, int c2, int lane)
{
    const int n = base + lane;
    bool ok = false;
    if (n < cl.N) {
        int mov_g = cl.free_g[n], mov_c = cl.free_c[n];
        if (mov_g < g2 || mov_c < c2) {
            const int cnt = nl.cnt[n];
            for (int i = 0; i < cnt; ++i) {
                const int v = nl.jobs[size_t(n) * nl.Gn + i];
                if (rl_pinned(roles[v])) continue;
                const uint32_t pk = hotA[v].packed;
                mov_g += sp.g_levels[pk_gi(pk)]; mov_c += sp.c_levels[pk_ci(pk)];
            }
        }
        ok = mov_g >= g2 && mov_c >= c2;
    }
    return __ballot_sync(0xffffffffu, ok);
}

// Lowest slope the single-node jobs of node n offer for GPUs and for cores (+inf when nobody offers), and
// the GPUs and cores its unpinned single-node jobs hold.  An exchange whose first step has to reclaim a
// resource on n fails there unless the candidate's gain exceeds the lowest slope, and it can never take
// more than what those jobs hold.  Warp-wide.
__device__ void node_min_slopes(const Space &sp, const Cluster &cl, const NodeLists &nl, const float *__restrict__ cv,
                                const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                                const uint32_t *__restrict__ feas, const HotA *hotA, const HotB *hotB, const uint32_t *roles,
                                int n, int lane, float &ms_g, float &ms_c, int &held_g, int &held_c)
{
    const float inf = __int_as_float(0x7f800000);
    float s[2] = {inf, inf};
    int hg = 0, hc = 0;
    if (lane < nl.cnt[n]) {
        const int v = nl.jobs[size_t(n) * nl.Gn + lane];
        const uint32_t vr = roles[v];
        if (!rl_pinned(vr)) {
            JobRegs vs; vs.a = hotA[v]; vs.b = hotB[v];
            hg = sp.g_levels[pk_gi(vs.a.packed)]; hc = sp.c_levels[pk_ci(vs.a.packed)];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                Offer of = shrink_offer(sp, cv, cp, cg, v, vs, vr, r);
                if (of.ok && of.gi2 >= 0) {
                    JobRegs t = vs; NodeFree tf; tf.g = cl.free_g[n]; tf.c = cl.free_c[n]; tf.m = cl.free_m[n];
                    of.ok = take_on_node(sp, cv, cp, cg, feas, v, t, tf, n, true, of.gi2, of.ci2, false);
                }
                if (of.ok) s[r] = of.slope;
            }
        }
    }
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) {
        s[0] = fminf(s[0], __shfl_xor_sync(0xffffffffu, s[0], k));
        s[1] = fminf(s[1], __shfl_xor_sync(0xffffffffu, s[1], k));
    }
    ms_g = s[0]; ms_c = s[1];
    held_g = __reduce_add_sync(0xffffffffu, hg); held_c = __reduce_add_sync(0xffffffffu, hc);
}

// Exchange attempt of job j for (gi2, ci2) on node n; warp 0, all lanes.  cand[r] = j's gain per unit
// of resource r (<= 0: r may not be reclaimed); force: a guaranteed minimum is being placed.
// On success the states of j and of the shrunk jobs, node n's free amounts and its job list are
// updated; on failure nothing is.
__device__ bool exchange_warp(const Space &sp, Cluster &cl, NodeLists &nl, const float *__restrict__ cv,
                              const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                              const uint32_t *__restrict__ feas, HotA *hotA, HotB *hotB, uint32_t *roles,
                              int j, int gi2, int ci2, int n, bool force, float cand_g, float cand_c,
                              bool need_gain, int lane)
{
    const unsigned FULLM = 0xffffffffu;
    JobRegs js; js.a = hotA[j]; js.b = hotB[j];
    const int jgi = pk_gi(js.a.packed);
    const bool on_n = jgi >= 0 && sp.g_levels[jgi] <= sp.Gn && js.a.node == n;
    const int need_g = sp.g_levels[gi2] - (on_n ? sp.g_levels[jgi] : 0);
    const int need_c = sp.c_levels[ci2] - (on_n ? sp.c_levels[pk_ci(js.a.packed)] : 0);

    // lane i owns the i-th single-node job of the node (never j itself, never a pinned job)
    const int cnt = nl.cnt[n];
    int v = lane < cnt ? nl.jobs[size_t(n) * nl.Gn + lane] : -1;
    uint32_t vr = 0; JobRegs vs; vs.a.packed = 0; vs.a.node = -1; vs.a.gain_g = vs.a.gain_c = 0.f; vs.b.val = 0.f; vs.b.plan = -1; vs.b.f_level = -1; vs.b.w = 0.f;
    if (v >= 0) { vr = roles[v]; vs.a = hotA[v]; vs.b = hotB[v]; }
    const bool victim = v >= 0 && v != j && !rl_pinned(vr);
    bool touched = false;

    NodeFree nf; nf.g = cl.free_g[n]; nf.c = cl.free_c[n]; nf.m = cl.free_m[n];
    bool ok = true;
    int taken = 0;
    for (int r = 0; r < 2 && ok; ++r) {
        const int need = r == 0 ? need_g : need_c;
        const float cand = r == 0 ? cand_g : cand_c;
        while ((r == 0 ? nf.g : nf.c) < need) {
            if (!force && !(cand > 0.0f)) { ok = false; break; }
            Offer of; of.ok = false; of.slope = 0.0f; of.gi2 = -1; of.ci2 = 0;
            if (victim && pk_gi(vs.a.packed) >= 0) {
                of = shrink_offer(sp, cv, cp, cg, v, vs, vr, r);
                if (of.ok && of.gi2 >= 0) {          // does the smaller allocation fit its memory on the node?
                    JobRegs t = vs; NodeFree tf = nf;
                    of.ok = take_on_node(sp, cv, cp, cg, feas, v, t, tf, n, true, of.gi2, of.ci2, false);
                }
            }
            // warp argmin on (slope, job index)
            float bs = of.slope; int bj = of.ok ? v : 0x7fffffff;
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) {
                const float os = __shfl_xor_sync(FULLM, bs, s);
                const int oj = __shfl_xor_sync(FULLM, bj, s);
                const bool better = oj != 0x7fffffff && (bj == 0x7fffffff || os < bs || (os == bs && oj < bj));
                bs = better ? os : bs; bj = better ? oj : bj;
            }
            if (bj == 0x7fffffff) { ok = false; break; }
            if (!force && !(cand > bs)) { ok = false; break; }
            if (++taken > MAX_EXCHANGE_STEPS) { ok = false; break; }
            // the winner shrinks in its registers; everybody learns the node's new free amounts
            NodeFree nf2 = nf;
            if (v == bj && of.ok) {
                if (of.gi2 < 0) {                    // preempted: everything goes back to the node
                    const int gi = pk_gi(vs.a.packed), ci = pk_ci(vs.a.packed);
                    nf2.g += sp.g_levels[gi]; nf2.c += sp.c_levels[ci]; nf2.m += sp.m_levels[vs.b.f_level];
                    vs.a.packed = pack(-1, 0, -1, false, true, true);
                    vs.a.node = -1; vs.b.val = 0.0f; vs.b.plan = -1; vs.b.f_level = -1;
                } else {
                    take_on_node(sp, cv, cp, cg, feas, v, vs, nf2, n, true, of.gi2, of.ci2, false);
                    vs.a.packed = pack(pk_gi(vs.a.packed), pk_ci(vs.a.packed), -1, false, true, true);
                }
                vs.a.gain_g = 0.0f; vs.a.gain_c = 0.0f;
                touched = true;
            }
            const int src = __ffs(__ballot_sync(FULLM, v == bj && of.ok)) - 1;
            nf.g = __shfl_sync(FULLM, nf2.g, src);
            nf.c = __shfl_sync(FULLM, nf2.c, src);
            nf.m = __shfl_sync(FULLM, nf2.m, src);
        }
    }
    if (ok) {
        bool placed = false;
        if (lane == 0) placed = take_on_node(sp, cv, cp, cg, feas, j, js, nf, n, on_n, gi2, ci2, need_gain);
        ok = __shfl_sync(FULLM, int(placed), 0) != 0;
    }
    if (!ok) return false;

    // ---- commit: states, node, list -----------------------------------------------------------------
    if (touched) { hotA[v] = vs.a; hotB[v] = vs.b; }
    if (lane == 0) {
        hotA[j] = js.a; hotB[j] = js.b;
        cl.free_g[n] = nf.g; cl.free_c[n] = nf.c; cl.free_m[n] = nf.m;
    }
    // list of the node: the jobs still on it, then j if it is new here
    const bool still = v >= 0 && pk_gi(vs.a.packed) >= 0;
    const unsigned keep = __ballot_sync(FULLM, still);
    if (still) nl.jobs[size_t(n) * nl.Gn + __popc(keep & ((1u << lane) - 1u))] = v;
    if (lane == 0) {
        int c2 = __popc(keep);
        if (!on_n) { nl.jobs[size_t(n) * nl.Gn + c2] = j; c2 += 1; }
        nl.cnt[n] = c2;
    }
    __syncwarp();
    return true;
}

__global__ void __launch_bounds__(ROUND_THREADS, 1)
incremental_round_kernel(const __grid_constant__ Space sp, const rubick_job *__restrict__ jobs, int J,
                         const float *__restrict__ cv, const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                         const uint32_t *__restrict__ feas, int N, int max_steps,
                         const rubick_assignment *__restrict__ prev, const rubick_node *__restrict__ prev_nodes,
                         const rubick_reconf *__restrict__ reconf, float theta,
                         rubick_assignment *__restrict__ out, rubick_node *__restrict__ node_out,
                         int32_t *__restrict__ step_log, HotA *hotA, HotB *hotB, uint32_t *roles, int32_t *own_count,
                         int32_t *list_jobs, const int32_t *__restrict__ quota, int n_tenants,
                         uint32_t *__restrict__ status, int32_t *__restrict__ steps_out)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ IncrShared sh;
    __shared__ int32_t rem_q[2 * RUBICK_MAX_TENANTS];

    // shared layout: free_m [N] i64 | free_g [N] | free_c [N] | owner [N] | list counts [N] | ff [n_small * nC] |
    // min slopes [2][N] | dirty [N] | held [2][N]
    Cluster cl;
    cl.N = N;
    cl.free_m = reinterpret_cast<int64_t *>(smem_raw);
    cl.free_g = reinterpret_cast<int32_t *>(cl.free_m + N);
    cl.free_c = cl.free_g + N;
    cl.owner = cl.free_c + N;
    NodeLists nl;
    nl.cnt = cl.owner + N;
    nl.jobs = list_jobs;
    nl.Gn = sp.Gn;
    cl.ff = nl.cnt + N;
    const int n_ff = sp.n_small * sp.nC;
    float *ms_g = reinterpret_cast<float *>(cl.ff + n_ff);      // [N] lowest offered GPU slope on the node
    float *ms_c = ms_g + N;                                     // [N] same for cores
    int32_t *dirty = reinterpret_cast<int32_t *>(ms_c + N);     // [N] the node changed since its slopes were worked out
    int32_t *held_g = dirty + N;                                // [N] GPUs held by the node's unpinned single-node jobs
    int32_t *held_c = held_g + N;                               // [N] their cores

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mt = sp.nM - 1;

    // ---- carried state --------------------------------------------------------------------------------
    for (int n = tid; n < N; n += ROUND_THREADS) {
        cl.free_g[n] = sp.Gn; cl.free_c[n] = sp.Cn; cl.free_m[n] = sp.Mn; cl.owner[n] = -1; nl.cnt[n] = 0;
    }
    for (int j = tid; j < J; j += ROUND_THREADS) own_count[j] = 0;
    if (tid == 0) { sh.steps = 0; sh.capped = 0; sh.n_empty = N; sh.changed = 1; sh.batch = 0; }
    for (int i = tid; i < 2 * n_tenants; i += ROUND_THREADS) rem_q[i] = quota[i];
    __syncthreads();

    bool bad = false;
    for (int j = tid; j < J; j += ROUND_THREADS) {
        const rubick_job *jb = jobs + j;
        const int gmin = jb->gmin_idx;
        const bool guaranteed = gmin >= 0;
        const int c0 = max(jb->cmin_idx, 0);
        int min_gi = -1;
        if (guaranteed && gmin < sp.nG && c0 < sp.nC) {
            const size_t o = curve_idx(sp, j, gmin, c0, mt);
            if (__ldg(cp + o) >= 0) min_gi = level_of_g(sp, __ldg(cg + o));
        }
        const bool active = reconf ? reconf[j].active != 0 : true;
        HotA a; a.gain_g = 0.0f; a.gain_c = 0.0f; a.node = -1;
        a.packed = pack(-1, min(c0, sp.nC - 1), -1, false, false, false);
        HotB b; b.val = 0.0f; b.plan = -1; b.f_level = -1; b.w = jb->w;
        bool pinned = false;
        if (active && prev && prev[j].status == RUBICK_RUNNING) {
            const rubick_assignment pv = prev[j];
            const int gi = level_of_g(sp, pv.g), ci = level_of_c(sp, pv.c);
            const int k = pv.n_nodes;
            if (gi < 0 || ci < 0 || pv.plan < 0 || pv.plan >= sp.P || pv.first_node < 0 || pv.first_node >= N || k < 1
                || (k == 1 ? pv.g > sp.Gn : pv.g != k * sp.Gn) || pv.m_level < 0 || pv.m_level >= sp.nM
                || sp.m_levels[pv.m_level < 0 || pv.m_level >= sp.nM ? 0 : pv.m_level] != pv.m_bytes) {
                bad = true;
            } else {
                a.node = pv.first_node;
                a.packed = pack(gi, ci, -1, false, false, false);
                b.val = pv.thr; b.plan = pv.plan; b.f_level = pv.m_level;
                if (k == 1) {
                    const int n = pv.first_node;
                    atomicSub(&cl.free_g[n], pv.g); atomicSub(&cl.free_c[n], pv.c);
                    atomicAdd(reinterpret_cast<unsigned long long *>(&cl.free_m[n]), static_cast<unsigned long long>(-pv.m_bytes));
                    const int slot = atomicAdd(&nl.cnt[n], 1);
                    if (slot < sp.Gn) nl.jobs[size_t(n) * sp.Gn + slot] = j; else bad = true;
                }
                float t = 1.0f, dl = 0.0f; int nr = 0;
                if (reconf) { t = reconf[j].T; dl = reconf[j].delta; nr = reconf[j].n_reconf; }
                const bool pass = t > 0.0f && __fdiv_rn(__fsub_rn(t, __fmul_rn(float(nr + 1), dl)), t) > theta;
                pinned = !pass;
            }
        }
        hotA[j] = a; hotB[j] = b;
        roles[j] = uint32_t(min_gi + 1) | (uint32_t(min(c0, 127)) << 6) | (uint32_t(guaranteed) << 13) | (uint32_t(pinned) << 14)
                   | (uint32_t(active) << 15);
    }
    __syncthreads();
    // whole nodes of multi-node jobs, as the previous round left them
    if (prev && prev_nodes)
        for (int n = tid; n < N; n += ROUND_THREADS) {
            const int j = prev_nodes[n].owner;
            if (j < 0) continue;
            if (j >= J) { bad = true; continue; }
            const int gi = pk_gi(hotA[j].packed);
            if (gi < 0 || sp.g_levels[gi] <= sp.Gn) continue;          // not running any more, or not a multi-node job
            const int k = sp.g_levels[gi] >> sp.log2Gn;
            const int c = sp.c_levels[pk_ci(hotA[j].packed)];
            const int64_t m = sp.m_levels[hotB[j].f_level];
            cl.free_g[n] -= sp.Gn; cl.free_c[n] -= (c + k - 1) / k; cl.free_m[n] -= cdiv64(m, k);
            cl.owner[n] = j;
            atomicAdd(&own_count[j], 1);
        }
    __syncthreads();
    for (int j = tid; j < J; j += ROUND_THREADS) {
        const int gi = pk_gi(hotA[j].packed);
        if (gi >= 0 && sp.g_levels[gi] > sp.Gn && own_count[j] != (sp.g_levels[gi] >> sp.log2Gn)) bad = true;
        const uint32_t r = roles[j];
        if (n_tenants > 0 && gi >= 0 && rl_guaranteed(r) && rl_min_gi(r) >= 0) {
            const int tn = jobs[j].tenant;
            if (tn >= 0 && tn < n_tenants) {
                atomicSub(&rem_q[2 * tn], sp.g_levels[rl_min_gi(r)]);
                atomicSub(&rem_q[2 * tn + 1], sp.c_levels[rl_min_ci(r)]);
            }
        }
    }
    for (int n = tid; n < N; n += ROUND_THREADS)
        if (cl.free_g[n] < 0 || cl.free_c[n] < 0 || cl.free_m[n] < 0) bad = true;
    if (__syncthreads_or(bad)) {                 // the previous state does not fit the grid or the cluster
        if (tid == 0) { atomicOr(status, DS_BAD_PREV); *steps_out = 0; }
        return;
    }

    // ---- Phase A: queued guaranteed jobs at their minimum, in job order (warp 0) --------------------------
    if (warp == 0) {
        int n_empty = 0;
        for (int nb = 0; nb < N; nb += 32) {
            const int n = nb + lane;
            n_empty += __popc(__ballot_sync(0xffffffffu, n < N && cl.free_g[n] == sp.Gn));
        }
        for (int base = 0; base < J; base += 32) {
            const int jj = base + lane;
            bool want = false;
            if (jj < J) { const uint32_t r = roles[jj]; want = rl_active(r) && rl_guaranteed(r) && pk_gi(hotA[jj].packed) < 0; }
            unsigned todo = __ballot_sync(0xffffffffu, want);
            while (todo) {
                const int j = base + __ffs(todo) - 1;
                todo &= todo - 1;
                const uint32_t r = roles[j];
                HotA a = hotA[j]; HotB b = hotB[j];
                a.packed = pack(-1, pk_ci(a.packed), -1, true, false, false);          // pending until placed
                if (lane == 0) hotA[j] = a;
                __syncwarp();
                const int gi = rl_min_gi(r), cmin = rl_min_ci(r);
                if (gi < 0) continue;
                const int tn = jobs[j].tenant;
                if (n_tenants > 0) {
                    if (tn < 0 || tn >= n_tenants) continue;
                    if (rem_q[2 * tn] < sp.g_levels[gi] || rem_q[2 * tn + 1] < sp.c_levels[cmin]) continue;
                }
                bool placed = commit_warp(sp, cl, n_empty, cv, cp, cg, feas, j, a, b, gi, cmin, false, lane);
                if (placed) {
                    if (lane == 0) {
                        hotA[j] = a; hotB[j] = b;
                        if (sp.g_levels[gi] <= sp.Gn) list_add(nl, a.node, j);
                    }
                    __syncwarp();
                } else if (sp.g_levels[gi] <= sp.Gn) {
                    for (int nb = 0; nb < N && !placed; nb += 32) {
                        unsigned todo2 = nodes_could_serve(sp, cl, nl, hotA, roles, nb, sp.g_levels[gi], sp.c_levels[cmin], lane);
                        while (todo2 && !placed) {
                            const int n = nb + __ffs(todo2) - 1;
                            todo2 &= todo2 - 1;
                            placed = exchange_warp(sp, cl, nl, cv, cp, cg, feas, hotA, hotB, roles, j, gi, cmin, n, true, 0.0f, 0.0f, false, lane);
                        }
                    }
                }
                if (placed) {
                    if (lane == 0 && n_tenants > 0) { rem_q[2 * tn] -= sp.g_levels[gi]; rem_q[2 * tn + 1] -= sp.c_levels[cmin]; }
                    __syncwarp();
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

    // gains of every job that may still grow
    for (int j = tid; j < J; j += ROUND_THREADS) {
        HotA a = hotA[j];
        const uint32_t r = roles[j];
        if (!rl_active(r) || rl_pinned(r) || pk_pending(a.packed)) continue;
        const bool fz_g = pk_fz_g(a.packed), fz_c = pk_fz_c(a.packed);       // shrunk while a minimum was placed
        const Gains gn = job_gains(sp, cv, j, hotB[j].w, pk_gi(a.packed), pk_ci(a.packed), hotB[j].val);
        a.gain_g = fz_g ? 0.0f : gn.gain_g; a.gain_c = fz_c ? 0.0f : gn.gain_c;
        a.packed = pack(pk_gi(a.packed), pk_ci(a.packed), gn.next_g, false, fz_g, fz_c);
        hotA[j] = a;
    }
    __syncthreads();

    // ---- Phase B ---------------------------------------------------------------------------------------------
    for (int n = tid; n < N; n += ROUND_THREADS) dirty[n] = 1;
    const float inf = __int_as_float(0x7f800000);
    // With a step log every attempt is taken one at a time.  Without one, candidates whose exchange cannot
    // get past its first step are frozen in bulk (same allocation, same step count).
    const bool bulk = step_log == nullptr;
    __syncthreads();
    for (;;) {
        if (sh.changed) {
            // an increment of (g, c) on one node fits somewhere exactly when the most free cores among the nodes
            // with at least g free GPUs reach c; the table only has to say "fits" (>= 0) or not
            for (int g = tid; g <= sp.Gn; g += ROUND_THREADS) sh.most_c[g] = -1;
            if (tid == 0) sh.n_empty = 0;
            __syncthreads();
            for (int n = tid; n < N; n += ROUND_THREADS) {
                const int fg = cl.free_g[n], fc = cl.free_c[n];
                for (int g = 1; g <= fg; ++g) atomicMax(&sh.most_c[g], fc);
                if (fg == sp.Gn) atomicAdd(&sh.n_empty, 1);
            }
            __syncthreads();
            for (int e = tid; e < n_ff; e += ROUND_THREADS) {
                const int gi = e / sp.nC, ci = e - gi * sp.nC;
                cl.ff[e] = sh.most_c[sp.g_levels[gi]] >= sp.c_levels[ci] ? 0 : -1;
            }
        }
        __syncthreads();

        // best increment that fits free resources (keys 0, 1) and best increment at all (keys 2, 3), GPU / CPU
        const int n_empty = sh.n_empty;
        unsigned long long best[4] = {0ull, 0ull, 0ull, 0ull};
        for (int j = tid; j < J; j += ROUND_THREADS) {
            const HotA a = hotA[j];
            const unsigned long long kg = (static_cast<unsigned long long>(__float_as_uint(a.gain_g)) << 32) | (0xffffffffu - uint32_t(j));
            const unsigned long long kc = (static_cast<unsigned long long>(__float_as_uint(a.gain_c)) << 32) | (0xffffffffu - uint32_t(j));
            const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
            if (a.gain_g > 0.0f) {
                if (kg > best[2]) best[2] = kg;
                if (kg > best[0] && placeable(sp, cl, n_empty, gi, ci, a.node, pk_next_gi(a.packed), ci)) best[0] = kg;
            }
            if (a.gain_c > 0.0f) {
                if (kc > best[3]) best[3] = kc;
                if (kc > best[1] && placeable(sp, cl, n_empty, gi, ci, a.node, gi, ci + 1)) best[1] = kc;
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) {
                const unsigned long long o = __shfl_xor_sync(0xffffffffu, best[q], s);
                best[q] = o > best[q] ? o : best[q];
            }
            if (lane == 0) sh.red[q][warp] = best[q];
        }
        __syncthreads();
        if (warp == 0) {
            unsigned long long b4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                b4[q] = sh.red[q][lane];
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) {
                    const unsigned long long o = __shfl_xor_sync(0xffffffffu, b4[q], s);
                    b4[q] = o > b4[q] ? o : b4[q];
                }
            }
            int which = -1;
            for (int q = 0; q < 4 && which < 0; ++q) if (b4[q]) which = q;
            if (lane == 0) {
                sh.which = which;
                sh.sel_j = which >= 0 ? int(0xffffffffu - uint32_t(b4[which])) : -1;
                sh.batch = bulk && which >= 2;
            }
        }
        __syncthreads();

        if (sh.batch) {
            // (a) lowest offered slopes of the nodes that changed
            for (int n = warp; n < N; n += ROUND_WARPS)
                if (dirty[n]) {
                    float g0, c0; int hg, hc;
                    node_min_slopes(sp, cl, nl, cv, cp, cg, feas, hotA, hotB, roles, n, lane, g0, c0, hg, hc);
                    if (lane == 0) { ms_g[n] = g0; ms_c[n] = c0; held_g[n] = hg; held_c[n] = hc; dirty[n] = 0; }
                }
            __syncthreads();
            // (b) over all nodes: lowest slopes, most free GPUs / cores
            {
                float lg = inf, lc = inf; int fg = 0, fc = 0;
                for (int n = tid; n < N; n += ROUND_THREADS) {
                    lg = fminf(lg, ms_g[n]); lc = fminf(lc, ms_c[n]);
                    fg = max(fg, cl.free_g[n]); fc = max(fc, cl.free_c[n]);
                }
#pragma unroll
                for (int k = 16; k > 0; k >>= 1) {
                    lg = fminf(lg, __shfl_xor_sync(0xffffffffu, lg, k)); lc = fminf(lc, __shfl_xor_sync(0xffffffffu, lc, k));
                    fg = max(fg, __shfl_xor_sync(0xffffffffu, fg, k)); fc = max(fc, __shfl_xor_sync(0xffffffffu, fc, k));
                }
                if (lane == 0) { sh.redf[0][warp] = lg; sh.redf[1][warp] = lc; sh.redi[0][warp] = fg; sh.redi[1][warp] = fc; }
                __syncthreads();
                if (warp == 0) {
                    lg = sh.redf[0][lane]; lc = sh.redf[1][lane]; fg = sh.redi[0][lane]; fc = sh.redi[1][lane];
#pragma unroll
                    for (int k = 16; k > 0; k >>= 1) {
                        lg = fminf(lg, __shfl_xor_sync(0xffffffffu, lg, k)); lc = fminf(lc, __shfl_xor_sync(0xffffffffu, lc, k));
                        fg = max(fg, __shfl_xor_sync(0xffffffffu, fg, k)); fc = max(fc, __shfl_xor_sync(0xffffffffu, fc, k));
                    }
                    if (lane == 0) { sh.min_slope[0] = lg; sh.min_slope[1] = lc; sh.max_free[0] = fg; sh.max_free[1] = fc; }
                }
                __syncthreads();
            }
            // (c) a candidate is hopeless when its exchange is sure to fail at the first step: no node (its own
            // node, for a running job) offers the resource below its gain.  Best candidate that is not hopeless:
            const float all_g = sh.min_slope[0];
            const int most_g = sh.max_free[0];
            auto hopeless = [&](int j, const HotA &a, int type) -> bool {
                const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
                const int gi2 = type == 0 ? pk_next_gi(a.packed) : gi;
                if (sp.g_levels[gi2] > sp.Gn) return true;              // increments above one node never exchange
                if (gi >= 0) {
                    if (sp.g_levels[gi] > sp.Gn) return true;
                    return type == 0 ? !(a.gain_g > ms_g[a.node]) : !(a.gain_c > ms_c[a.node]);
                }
                // a queued job reclaims GPUs first: where every node lacks them, the first step decides.  (Its
                // cores come second and may be freed by a preemption of the GPU phase: no shortcut there.)
                return most_g < sp.g_levels[gi2] && !(a.gain_g > all_g);
            };
            unsigned long long live[2] = {0ull, 0ull};
            for (int j = tid; j < J; j += ROUND_THREADS) {
                const HotA a = hotA[j];
                const unsigned long long kg = (static_cast<unsigned long long>(__float_as_uint(a.gain_g)) << 32) | (0xffffffffu - uint32_t(j));
                const unsigned long long kc = (static_cast<unsigned long long>(__float_as_uint(a.gain_c)) << 32) | (0xffffffffu - uint32_t(j));
                if (a.gain_g > 0.0f && kg > live[0] && !hopeless(j, a, 0)) live[0] = kg;
                if (a.gain_c > 0.0f && kc > live[1] && !hopeless(j, a, 1)) live[1] = kc;
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
#pragma unroll
                for (int k = 16; k > 0; k >>= 1) {
                    const unsigned long long o = __shfl_xor_sync(0xffffffffu, live[q], k);
                    live[q] = o > live[q] ? o : live[q];
                }
                if (lane == 0) sh.red[q][warp] = live[q];
            }
            __syncthreads();
            unsigned long long lv[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                lv[q] = sh.red[q][lane];
#pragma unroll
                for (int k = 16; k > 0; k >>= 1) {
                    const unsigned long long o = __shfl_xor_sync(0xffffffffu, lv[q], k);
                    lv[q] = o > lv[q] ? o : lv[q];
                }
            }
            __syncthreads();
            // (d) hopeless candidates that come before it (GPU increments before CPU increments, larger key first)
            // would each be tried, fail and be frozen: count them, freeze them
            const int live_type = lv[0] ? 0 : (lv[1] ? 1 : 2);
            int mine = 0;
            for (int j = tid; j < J; j += ROUND_THREADS) {
                HotA a = hotA[j];
                const unsigned long long kg = (static_cast<unsigned long long>(__float_as_uint(a.gain_g)) << 32) | (0xffffffffu - uint32_t(j));
                const unsigned long long kc = (static_cast<unsigned long long>(__float_as_uint(a.gain_c)) << 32) | (0xffffffffu - uint32_t(j));
                bool fg = false, fc = false;
                if (a.gain_g > 0.0f && (live_type > 0 || kg > lv[0]) && hopeless(j, a, 0)) fg = true;
                if (a.gain_c > 0.0f && live_type > 0 && (live_type > 1 || kc > lv[1]) && hopeless(j, a, 1)) fc = true;
                if (fg || fc) {
                    mine += int(fg) + int(fc);
                    if (fg) a.gain_g = 0.0f;
                    if (fc) a.gain_c = 0.0f;
                    a.packed = pack(pk_gi(a.packed), pk_ci(a.packed), pk_next_gi(a.packed), false, pk_fz_g(a.packed) || fg, pk_fz_c(a.packed) || fc);
                    hotA[j] = a;
                }
            }
            mine = __reduce_add_sync(0xffffffffu, mine);
            if (lane == 0) sh.redi[2][warp] = mine;
            __syncthreads();
            if (warp == 0) {
                const int frozen = __reduce_add_sync(0xffffffffu, sh.redi[2][lane]);
                if (lane == 0) {
                    if (sh.steps + frozen > max_steps) {               // the cap falls inside the run of failures
                        sh.steps = max_steps; sh.capped = 1; sh.sel_j = -1; sh.which = -1;
                    } else {
                        sh.steps += frozen;
                        sh.which = live_type < 2 ? 2 + live_type : -1;
                        sh.sel_j = live_type < 2 ? int(0xffffffffu - uint32_t(lv[live_type])) : -1;
                    }
                }
            }
            __syncthreads();
        }

        if (warp == 0) {
            const int which = sh.which;
            int sel_j = sh.sel_j;
            if (sel_j >= 0 && sh.steps >= max_steps) { if (lane == 0) sh.capped = 1; sel_j = -1; }
            bool ok = false;
            if (sel_j >= 0) {
                const int j = sel_j, type = which & 1;
                const bool by_exchange = which >= 2;
                HotA a = hotA[j]; HotB b = hotB[j];
                const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
                const int gi2 = type == 0 ? pk_next_gi(a.packed) : gi;
                const int ci2 = type == 0 ? ci : ci + 1;
                const float gain = type == 0 ? a.gain_g : a.gain_c;
                const int old_node = a.node;
                const bool was_single = gi >= 0 && sp.g_levels[gi] <= sp.Gn;
                if (!by_exchange) {
                    ok = commit_warp(sp, cl, n_empty, cv, cp, cg, feas, j, a, b, gi2, ci2, true, lane);
                    if (ok && lane == 0) {
                        if (was_single) { list_remove(nl, old_node, j); dirty[old_node] = 1; }
                        if (sp.g_levels[gi2] <= sp.Gn) { list_add(nl, a.node, j); dirty[a.node] = 1; }
                    }
                    __syncwarp();
                } else if (sp.g_levels[gi2] <= sp.Gn) {
                    // what j gains per unit of each resource it would take from others: a running job asks
                    // only for the resource of its increment; a queued job pre-allocates GPUs and cores
                    // together, so its value counts per GPU and per core
                    float cand_g = type == 0 ? gain : 0.0f, cand_c = type == 1 ? gain : 0.0f;
                    if (gi >= 0) {
                        if (sp.g_levels[gi] <= sp.Gn)
                            ok = exchange_warp(sp, cl, nl, cv, cp, cg, feas, hotA, hotB, roles, j, gi2, ci2, a.node, false, cand_g, cand_c, true, lane);
                    } else {
                        const float v2 = cv[curve_idx(sp, j, gi2, ci2, mt)];
                        cand_c = __fdiv_rn(__fsub_rn(__fmul_rn(b.w, v2), 0.0f), float(sp.c_levels[ci2]));
                        const int g2 = sp.g_levels[gi2], c2 = sp.c_levels[ci2];
                        for (int nb = 0; nb < N && !ok; nb += 32) {
                            unsigned todo;
                            if (bulk) {
                                // the per-node figures are fresh: enough free plus held amounts and, where GPUs
                                // are short, a first offer below the gain
                                const int n = nb + lane;
                                const bool worth = n < N && cl.free_g[n] + held_g[n] >= g2 && cl.free_c[n] + held_c[n] >= c2
                                                   && (cl.free_g[n] >= g2 || cand_g > ms_g[n]);
                                todo = __ballot_sync(0xffffffffu, worth);
                            } else {
                                todo = nodes_could_serve(sp, cl, nl, hotA, roles, nb, g2, c2, lane);
                            }
                            while (todo && !ok) {
                                const int n2 = nb + __ffs(todo) - 1;
                                todo &= todo - 1;
                                ok = exchange_warp(sp, cl, nl, cv, cp, cg, feas, hotA, hotB, roles, j, gi2, ci2, n2, false, cand_g, cand_c, true, lane);
                            }
                        }
                    }
                    if (ok) { a = hotA[j]; b = hotB[j]; if (lane == 0) dirty[a.node] = 1; }
                }
                bool fz_g = pk_fz_g(a.packed), fz_c = pk_fz_c(a.packed);
                if (!ok) { if (type == 0) fz_g = true; else fz_c = true; }
                const Gains gn = job_gains(sp, cv, j, b.w, pk_gi(a.packed), pk_ci(a.packed), b.val);
                a.gain_g = fz_g ? 0.0f : gn.gain_g;
                a.gain_c = fz_c ? 0.0f : gn.gain_c;
                a.packed = pack(pk_gi(a.packed), pk_ci(a.packed), gn.next_g, false, fz_g, fz_c);
                if (lane == 0) {
                    hotA[j] = a; hotB[j] = b;
                    if (step_log) step_log[sh.steps] = (j << 3) | (int(by_exchange) << 2) | (type << 1) | int(ok);
                    sh.steps += 1;
                }
            }
            if (lane == 0) { sh.sel_j = sel_j; sh.changed = ok ? 1 : 0; }
        }
        __syncthreads();
        if (sh.sel_j < 0) break;
    }

    // ---- results -----------------------------------------------------------------------------------------------
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

static size_t incr_smem(const Space &sp, int N)
{
    return (size_t(N) * 44 + size_t(sp.n_small) * sp.nC * 4 + 15) & ~size_t(15);
}

// scratch: HotA [J] | HotB [J] | roles [J] | whole-node counts [J] | node lists [N][Gn]
size_t incr_scratch_need(const Space &sp, int J, int N)
{
    return size_t(J) * (sizeof(HotA) + sizeof(HotB) + 8) + size_t(N) * sp.Gn * 4 + 64;
}

cudaError_t launch_round_incremental(const Space &sp, const rubick_job *d_jobs, int J, const float *d_cv, const int32_t *d_cp,
                                     const int32_t *d_cg, const uint32_t *d_feas, int N, int max_steps,
                                     const rubick_assignment *d_prev, const rubick_node *d_prev_nodes,
                                     const rubick_reconf *d_reconf, float theta, rubick_assignment *d_out,
                                     rubick_node *d_node_out, int32_t *d_step_log, void *d_scratch,
                                     const int32_t *d_quota, int n_tenants, uint32_t *d_status, int32_t *d_steps,
                                     cudaStream_t st)
{
    // a step raises a job by a level or freezes one (job, resource) pair, and a shrunk job never grows
    // again, so a round cannot take more steps than this; the clamp keeps the device loop bounded
    const long long natural = 2LL * J * (sp.nG + sp.nC + 2) + 1;
    if ((long long)max_steps > natural) max_steps = int(natural < 0x7fffffffLL ? natural : 0x7fffffffLL);
    const size_t smem = incr_smem(sp, N);
    cudaError_t e = cudaFuncSetAttribute(incremental_round_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(200 * 1024));
    if (e != cudaSuccess) return e;
    unsigned char *p = reinterpret_cast<unsigned char *>(d_scratch);
    HotA *ha = reinterpret_cast<HotA *>(p); p += size_t(J) * sizeof(HotA);
    HotB *hb = reinterpret_cast<HotB *>(p); p += size_t(J) * sizeof(HotB);
    uint32_t *roles = reinterpret_cast<uint32_t *>(p); p += size_t(J) * 4;
    int32_t *own = reinterpret_cast<int32_t *>(p); p += size_t(J) * 4;
    int32_t *lists = reinterpret_cast<int32_t *>(p);
    incremental_round_kernel<<<1, ROUND_THREADS, smem, st>>>(sp, d_jobs, J, d_cv, d_cp, d_cg, d_feas, N, max_steps, d_prev,
                                                             d_prev_nodes, d_reconf, theta, d_out, d_node_out, d_step_log,
                                                             ha, hb, roles, own, lists, d_quota, n_tenants, d_status, d_steps); count_launch();
    return cudaGetLastError();
}

}  // namespace rubick
