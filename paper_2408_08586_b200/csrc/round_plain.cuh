// Device helpers shared by the single-CTA round kernels (the plain greedy round and the incremental
// round): per-job scan state, gains, node state views, placement test and the warp-cooperative commit.
#pragma once

#include "rubick_internal.cuh"

namespace rubick {

constexpr int ROUND_THREADS = 1024;
constexpr int ROUND_WARPS = ROUND_THREADS / 32;

// scan state of one job (16 bytes)
struct HotA {
    float gain_g, gain_c;     // 0 = no candidate
    uint32_t packed;          // see pack()
    int32_t node;             // node of a single-node job, lowest node of a multi-node job, -1 if none
};
// the rest of a job's state (16 bytes)
struct HotB {
    float val;                // predicted throughput of the present allocation
    int32_t plan;
    int32_t f_level;          // host-memory level allocated (first feasible level of the plan)
    float w;
};

// packed: [5:0] present g level + 1 (0 = nothing held) | [12:6] c level (present, or where an
// unallocated job would start) | [18:13] target g level + 1 (0 = none) | [19] pending |
// [20] GPU increments frozen | [21] CPU increments frozen
__device__ __forceinline__ uint32_t pack(int gi, int ci, int next_gi, bool pending, bool fz_g, bool fz_c)
{
    return uint32_t(gi + 1) | (uint32_t(ci) << 6) | (uint32_t(next_gi + 1) << 13) | (uint32_t(pending) << 19)
           | (uint32_t(fz_g) << 20) | (uint32_t(fz_c) << 21);
}
__device__ __forceinline__ int pk_gi(uint32_t p) { return int(p & 63u) - 1; }
__device__ __forceinline__ int pk_ci(uint32_t p) { return int((p >> 6) & 127u); }
__device__ __forceinline__ int pk_next_gi(uint32_t p) { return int((p >> 13) & 63u) - 1; }
__device__ __forceinline__ bool pk_pending(uint32_t p) { return (p >> 19) & 1u; }
__device__ __forceinline__ bool pk_fz_g(uint32_t p) { return (p >> 20) & 1u; }
__device__ __forceinline__ bool pk_fz_c(uint32_t p) { return (p >> 21) & 1u; }

__device__ __forceinline__ size_t curve_idx(const Space &sp, int j, int gi, int ci, int mi)
{
    return ((size_t(j) * sp.nG + gi) * sp.nC + ci) * sp.nM + mi;
}

struct Gains { int next_g, next_c; float gain_g, gain_c; };

// One thread computes the gains of one job from the curve table.
__device__ inline Gains job_gains(const Space &sp, const float *__restrict__ cv, int j, float w, int gi, int ci, float val)
{
    Gains r; r.next_g = -1; r.next_c = -1; r.gain_g = 0.0f; r.gain_c = 0.0f;
    const int mt = sp.nM - 1;
    const bool alloc = gi >= 0;
    const float cur = alloc ? val : 0.0f;
    const float vcur = alloc ? __fmul_rn(w, cur) : 0.0f;
    for (int g2 = gi + 1; g2 < sp.nG; ++g2) {
        const float v = cv[curve_idx(sp, j, g2, ci, mt)];
        if (v > cur) {
            const float dg = float(sp.g_levels[g2] - (alloc ? sp.g_levels[gi] : 0));
            r.next_g = g2;
            r.gain_g = __fdiv_rn(__fsub_rn(__fmul_rn(w, v), vcur), dg);
            break;
        }
    }
    if (alloc && ci + 1 < sp.nC) {
        const float v = cv[curve_idx(sp, j, gi, ci + 1, mt)];
        const float dc = float(sp.c_levels[ci + 1] - sp.c_levels[ci]);
        const float gn = __fdiv_rn(__fsub_rn(__fmul_rn(w, v), vcur), dc);
        if (gn > 0.0f) { r.next_c = ci + 1; r.gain_c = gn; }
    }
    return r;
}

__device__ __forceinline__ int level_of_g(const Space &sp, int g)
{
    for (int i = 0; i < sp.nG; ++i) if (sp.g_levels[i] == g) return i;
    return -1;
}
__device__ __forceinline__ int level_of_c(const Space &sp, int c)
{
    for (int i = 0; i < sp.nC; ++i) if (sp.c_levels[i] == c) return i;
    return -1;
}

struct Cluster {           // views into shared memory
    int32_t *free_g, *free_c, *owner;
    int64_t *free_m;
    int32_t *ff;           // [n_small][nC] first node that fits the whole job, -1 if none
    int N;
};

__device__ __forceinline__ int64_t cdiv64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Can (g level gi2, c level ci2) be placed for a job that holds (gi, ci) on `node`?
__device__ __forceinline__ bool placeable(const Space &sp, const Cluster &cl, int n_empty, int gi, int ci, int node,
                                          int gi2, int ci2)
{
    const int g2 = sp.g_levels[gi2], c2 = sp.c_levels[ci2];
    const bool alloc = gi >= 0;
    const int g = alloc ? sp.g_levels[gi] : 0, c = alloc ? sp.c_levels[ci] : 0;
    if (g2 <= sp.Gn) {
        if (alloc && cl.free_g[node] >= g2 - g && cl.free_c[node] >= c2 - c) return true;
        return cl.ff[gi2 * sp.nC + ci2] >= 0;
    }
    const int k2 = g2 >> sp.log2Gn;
    if ((c2 + k2 - 1) / k2 > sp.Cn) return false;
    if (alloc && g >= sp.Gn) { const int k = g >> sp.log2Gn; return n_empty >= k2 - k; }
    const int empty = n_empty + ((alloc && cl.free_g[node] + g == sp.Gn) ? 1 : 0);
    return empty >= k2;
}

// warp-cooperative: first node with at least g free GPUs and c free cores, -1 if none
__device__ inline int first_fit_warp(const Cluster &cl, int g, int c, int lane)
{
    for (int base = 0; base < cl.N; base += 32) {
        const int n = base + lane;
        const bool ok = n < cl.N && cl.free_g[n] >= g && cl.free_c[n] >= c;
        const unsigned b = __ballot_sync(0xffffffffu, ok);
        if (b) return base + __ffs(b) - 1;
    }
    return -1;
}

struct RoundShared {
    unsigned long long red[2][ROUND_WARPS];
    int n_empty;
    int sel_j, sel_type;
    int steps, capped;
};

// Commit job j to (gi2, ci2); executed by warp 0 (all lanes).  Returns true when the allocation
// was made.  need_gain: the new value must strictly exceed the present one.
__device__ inline bool commit_warp(const Space &sp, Cluster &cl, int n_empty, const float *__restrict__ cv,
                            const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                            const uint32_t *__restrict__ feas, int j, HotA &ha, HotB &hb, int gi2, int ci2,
                            bool need_gain, int lane)
{
    const int gi = pk_gi(ha.packed), ci = pk_ci(ha.packed);
    const bool alloc = gi >= 0;
    const int g = alloc ? sp.g_levels[gi] : 0, c = alloc ? sp.c_levels[ci] : 0;
    const int64_t m_cur = alloc ? sp.m_levels[hb.f_level] : 0;
    const int g2 = sp.g_levels[gi2], c2 = sp.c_levels[ci2];
    const int k = alloc ? max(g >> sp.log2Gn, 1) : 0;

    // ---- placement -----------------------------------------------------------------------------
    int k2 = 1, target = -1, need_new = 0;
    bool stay = false;
    if (g2 <= sp.Gn) {
        if (alloc && cl.free_g[ha.node] >= g2 - g && cl.free_c[ha.node] >= c2 - c) { stay = true; target = ha.node; }
        else target = first_fit_warp(cl, g2, c2, lane);
        if (target < 0) return false;
    } else {
        k2 = g2 >> sp.log2Gn;
        if ((c2 + k2 - 1) / k2 > sp.Cn) return false;
        if (alloc && g >= sp.Gn) { stay = true; need_new = k2 - k; if (n_empty < need_new) return false; }
        else {
            need_new = k2;
            const int empty = n_empty + ((alloc && cl.free_g[ha.node] + g == sp.Gn) ? 1 : 0);
            if (empty < need_new) return false;
        }
    }

    // ---- host-memory level that fits the target, curve lookup, memory of the plan ---------------
    const int64_t avail = k2 > 1 ? sp.Mn : cl.free_m[target] + ((stay && alloc) ? m_cur : 0);
    const bool fits = lane < sp.nM && cdiv64(sp.m_levels[lane < sp.nM ? lane : 0], k2) <= avail;
    const unsigned fb = __ballot_sync(0xffffffffu, fits);
    if (!fb) return false;
    const int mi = 31 - __clz(fb);
    const size_t o = curve_idx(sp, j, gi2, ci2, mi);
    const float v = __ldg(cv + o);
    const int plan = __ldg(cp + o), gu = __ldg(cg + o);
    if (plan < 0 || plan >= sp.P || !(v > 0.0f) || gu != g2) return false;
    if (need_gain && alloc && !(v > hb.val)) return false;
    const uint32_t word = __ldg(feas + size_t(j) * sp.P + plan);
    const int f = __ffs(word) - 1;
    if (f < 0 || f > mi) return false;
    const int64_t m2 = sp.m_levels[f];

    // ---- node bookkeeping ------------------------------------------------------------------------
    int first = -1;
    if (k2 == 1) {
        if (lane == 0) {
            if (alloc) { cl.free_g[ha.node] += g; cl.free_c[ha.node] += c; cl.free_m[ha.node] += m_cur; }
            cl.free_g[target] -= g2; cl.free_c[target] -= c2; cl.free_m[target] -= m2;
        }
        first = target;
    } else {
        const int cs2 = (c2 + k2 - 1) / k2;
        const int64_t ms2 = cdiv64(m2, k2);
        if (stay) {
            // whole nodes already held keep their GPUs; only the core / memory shares change
            const int cs1 = (c + k - 1) / k;
            const int64_t ms1 = cdiv64(m_cur, k);
            if (k == 1) {
                if (lane == 0) { cl.free_c[ha.node] += c - cs2; cl.free_m[ha.node] += m_cur - ms2; cl.owner[ha.node] = j; }
            } else {
                for (int n = lane; n < cl.N; n += 32)
                    if (cl.owner[n] == j) { cl.free_c[n] += cs1 - cs2; cl.free_m[n] += ms1 - ms2; }
            }
            first = ha.node;
        } else if (alloc && lane == 0) {
            cl.free_g[ha.node] += g; cl.free_c[ha.node] += c; cl.free_m[ha.node] += m_cur;
        }
        __syncwarp();
        int taken = 0;
        for (int base = 0; base < cl.N && taken < need_new; base += 32) {
            const int n = base + lane;
            const bool empty = n < cl.N && cl.free_g[n] == sp.Gn;
            const unsigned b = __ballot_sync(0xffffffffu, empty);
            const int rank = __popc(b & ((1u << lane) - 1u));
            if (empty && taken + rank < need_new) {
                cl.free_g[n] = 0; cl.free_c[n] -= cs2; cl.free_m[n] -= ms2; cl.owner[n] = j;
            }
            if (b) { const int lowest = base + __ffs(b) - 1; if (first < 0 || lowest < first) first = lowest; }
            taken += __popc(b);
        }
    }
    __syncwarp();
    ha.node = first;
    ha.packed = pack(gi2, ci2, -1, false, pk_fz_g(ha.packed), pk_fz_c(ha.packed));
    hb.val = v; hb.plan = plan; hb.f_level = f;
    return true;
}

}  // namespace rubick
