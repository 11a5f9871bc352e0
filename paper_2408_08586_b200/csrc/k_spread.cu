// Greedy round with spread placement (paper Section 5.2 / Algorithm 1: a job's placement is a list of per-node
// allocations found node by node, the plan is chosen for the placement found; Section 4.1: groups whose GPUs sit on
// several nodes communicate at the inter-node bandwidth).
//
// Same step list as the plain round in k_sched.cu (guaranteed minima in job order, then the placeable increment
// with the largest positive GPU gain, CPU gain when no GPU increment is left, lowest job on ties), with one more
// way to place a job of at most one node's GPUs: when no node takes it whole, it is assembled from free pieces of
// a GPUs on several nodes (classes in the order given, nodes in index order), and the commit reads plan and value
// from that class's tables.  One persistent CTA; every step rescans all jobs against per-step tables (first fit
// per (GPU level, core level); per spread class, whether enough pieces can be found).  Increments that a node
// takes whole go through the plain round's warp-cooperative commit; everything that involves pieces is worked out
// by one thread, step by step as the rule is stated, since that is the rare case and correctness matters more
// than speed here.

#include "round_plain.cuh"

namespace rubick {

struct SpreadArgs {
    int nK;
    int32_t align[RUBICK_MAX_SPREAD_CLASSES];
    const float *cv[RUBICK_MAX_SPREAD_CLASSES];
    const int32_t *cp[RUBICK_MAX_SPREAD_CLASSES];
    const int32_t *cg[RUBICK_MAX_SPREAD_CLASSES];
    const uint32_t *feas[RUBICK_MAX_SPREAD_CLASSES];
};

__device__ __forceinline__ int64_t cdiv_i64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// what the scan needs per job beyond the plain round's state: class and pieces live in the caller's output arrays
struct SpreadView {
    int32_t *pieces;          // [J][RUBICK_MAX_PIECES] node << 8 | GPUs, -1 = unused
    int32_t *cls;             // [J]
    const uint8_t *sf;        // [nK][n_small][nC] enough free pieces for (class, GPU level, core level)?
};

// Can the increment to (gi2, ci2) be placed?  (the selection only counts increments that can)
__device__ bool placeable_spread(const Space &sp, const Cluster &cl, const SpreadArgs &S, const SpreadView &V, int n_empty,
                                 int j, int gi, int ci, int node, int gi2, int ci2)
{
    const int cls = gi >= 0 ? V.cls[j] : -1;
    if (cls < 0) {
        if (placeable(sp, cl, n_empty, gi, ci, node, gi2, ci2)) return true;
    } else {
        // a job that sits in pieces: more cores stay on its nodes when each has them; anything else is placed anew
        // from free resources (what it holds is not counted)
        const int g = sp.g_levels[gi], c = sp.c_levels[ci], g2 = sp.g_levels[gi2], c2 = sp.c_levels[ci2];
        const int a = S.align[cls];
        if (g2 == g) {
            const int extra = int(cdiv_i64(int64_t(c2) * a, g2) - cdiv_i64(int64_t(c) * a, g));
            bool fits = true;
            for (int i = 0; i < RUBICK_MAX_PIECES; ++i) {
                const int e = V.pieces[size_t(j) * RUBICK_MAX_PIECES + i];
                if (e < 0) break;
                if (cl.free_c[e >> 8] < extra * ((e & 255) / a)) fits = false;
            }
            if (fits) return true;
        }
        if (g2 <= sp.Gn) { if (cl.ff[gi2 * sp.nC + ci2] >= 0) return true; }
        else {
            const int k2 = g2 >> sp.log2Gn;
            return (c2 + k2 - 1) / k2 <= sp.Cn && n_empty >= k2;
        }
    }
    if (sp.g_levels[gi2] > sp.Gn) return false;
    for (int k = 0; k < S.nK; ++k)
        if (V.sf[(size_t(k) * sp.n_small + gi2) * sp.nC + ci2]) return true;
    return false;
}

// One thread: place job j at (gi2, ci2) in a way that involves pieces -- the job sits in pieces now, or no node
// takes the increment whole and it has to be assembled from pieces.  Mirrors the rule as stated: find the
// placement, pick the memory level, read the tables of the placement's class, give back the old allocation, take
// the new one.  Returns true when the allocation was made.
__device__ bool commit_pieces(const Space &sp, Cluster &cl, const SpreadArgs &S, const SpreadView &V, int n_empty,
                              const float *__restrict__ cv, const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                              const uint32_t *__restrict__ feas, int j, HotA &ha, HotB &hb, int gi2, int ci2, bool need_gain)
{
    const int gi = pk_gi(ha.packed), ci = pk_ci(ha.packed);
    const bool alloc = gi >= 0;
    const int cls = alloc ? V.cls[j] : -1;
    const bool spread = cls >= 0;
    const int g = alloc ? sp.g_levels[gi] : 0, c = alloc ? sp.c_levels[ci] : 0;
    const int64_t m_cur = alloc ? sp.m_levels[hb.f_level] : 0;
    const int g2 = sp.g_levels[gi2], c2 = sp.c_levels[ci2];
    int32_t *mine = V.pieces + size_t(j) * RUBICK_MAX_PIECES;

    // ---- placement ---------------------------------------------------------------------------------------
    enum { ONE_NODE, PIECES, WHOLE_NODES } kind = ONE_NODE;
    int target = -1, k2 = 1, new_cls = -1, np = 0;
    bool stay = false;
    int pn[RUBICK_MAX_PIECES], pq[RUBICK_MAX_PIECES];
    if (g2 <= sp.Gn) {
        if (spread && g2 == g) {
            const int a = S.align[cls];
            const int extra = int(cdiv_i64(int64_t(c2) * a, g2) - cdiv_i64(int64_t(c) * a, g));
            bool fits = true;
            for (int i = 0; i < RUBICK_MAX_PIECES && mine[i] >= 0; ++i) {
                pn[np] = mine[i] >> 8; pq[np] = (mine[i] & 255) / a; ++np;
                if (cl.free_c[pn[np - 1]] < extra * pq[np - 1]) fits = false;
            }
            if (fits) { kind = PIECES; stay = true; new_cls = cls; }
        }
        if (!stay) {
            for (int n = 0; n < cl.N && target < 0; ++n)
                if (cl.free_g[n] >= g2 && cl.free_c[n] >= c2) target = n;
            if (target < 0) {
                for (int k = 0; k < S.nK && new_cls < 0; ++k) {
                    const int a = S.align[k];
                    if (a <= 0 || g2 % a != 0 || g2 <= a) continue;
                    const int want = g2 / a, cpp = int(cdiv_i64(int64_t(c2) * a, g2));
                    int left = want;
                    np = 0;
                    for (int n = 0; n < cl.N && left > 0 && np < RUBICK_MAX_PIECES; ++n) {
                        int q = min(cl.free_g[n] / a, cl.free_c[n] / cpp);
                        if (q <= 0) continue;
                        if (q > left) q = left;
                        pn[np] = n; pq[np] = q; ++np; left -= q;
                    }
                    if (left == 0) { new_cls = k; kind = PIECES; }
                }
                if (new_cls < 0) return false;
            }
        }
    } else {
        // above one node: whole nodes from the empty ones (what a job in pieces holds is not counted)
        kind = WHOLE_NODES;
        k2 = g2 >> sp.log2Gn;
        if ((c2 + k2 - 1) / k2 > sp.Cn || n_empty < k2) return false;
    }

    // ---- host-memory level that fits the placement, tables of its class, memory of the plan ---------------
    int mi = -1;
    if (kind == PIECES) {
        const int a = S.align[new_cls];
        const int64_t own = (stay && alloc) ? cdiv_i64(m_cur * a, g) : 0;
        for (int i = 0; i < sp.nM; ++i) {
            const int64_t mpp = cdiv_i64(sp.m_levels[i] * a, g2);
            bool fits = true;
            for (int q = 0; q < np; ++q) if (mpp * pq[q] > cl.free_m[pn[q]] + own * pq[q]) fits = false;
            if (fits) mi = i;
        }
    } else {
        const int64_t avail = kind == WHOLE_NODES ? sp.Mn : cl.free_m[target];
        for (int i = 0; i < sp.nM; ++i) if (cdiv_i64(sp.m_levels[i], k2) <= avail) mi = i;
    }
    if (mi < 0) return false;
    const size_t o = curve_idx(sp, j, gi2, ci2, mi);
    const float *tv = kind == PIECES ? S.cv[new_cls] : cv;
    const int32_t *tp = kind == PIECES ? S.cp[new_cls] : cp, *tg = kind == PIECES ? S.cg[new_cls] : cg;
    const uint32_t *tf = kind == PIECES ? S.feas[new_cls] : feas;
    const float v = tv[o];
    const int plan = tp[o], gu = tg[o];
    if (plan < 0 || plan >= sp.P || !(v > 0.0f) || gu != g2) return false;
    if (need_gain && alloc && !(v > hb.val)) return false;
    const int f = __ffs(tf[size_t(j) * sp.P + plan]) - 1;
    if (f < 0 || f > mi) return false;
    const int64_t m2 = sp.m_levels[f];

    // ---- give back what the job holds, take the new placement ----------------------------------------------
    if (alloc) {
        if (spread) {
            const int a = S.align[cls];
            const int64_t cpp = cdiv_i64(int64_t(c) * a, g), mpp = cdiv_i64(m_cur * a, g);
            for (int i = 0; i < RUBICK_MAX_PIECES && mine[i] >= 0; ++i) {
                const int n = mine[i] >> 8, q = (mine[i] & 255) / a;
                cl.free_g[n] += a * q; cl.free_c[n] += int(cpp) * q; cl.free_m[n] += mpp * q;
            }
        } else {
            // a job on one node (jobs on whole nodes never get here: their increments lead above a node)
            cl.free_g[ha.node] += g; cl.free_c[ha.node] += c; cl.free_m[ha.node] += m_cur;
        }
    }
    for (int i = 0; i < RUBICK_MAX_PIECES; ++i) mine[i] = -1;
    int first = -1;
    if (kind == PIECES) {
        const int a = S.align[new_cls];
        const int64_t cpp = cdiv_i64(int64_t(c2) * a, g2), mpp = cdiv_i64(m2 * a, g2);
        for (int i = 0; i < np; ++i) {
            const int n = pn[i];
            cl.free_g[n] -= a * pq[i]; cl.free_c[n] -= int(cpp) * pq[i]; cl.free_m[n] -= mpp * pq[i];
            mine[i] = (n << 8) | (a * pq[i]);
        }
        first = pn[0];
    } else if (kind == ONE_NODE) {
        cl.free_g[target] -= g2; cl.free_c[target] -= c2; cl.free_m[target] -= m2;
        first = target;
    } else {
        const int cs2 = (c2 + k2 - 1) / k2;
        const int64_t ms2 = cdiv_i64(m2, k2);
        int taken = 0;
        for (int n = 0; n < cl.N && taken < k2; ++n)
            if (cl.owner[n] != j && cl.free_g[n] == sp.Gn) {
                cl.free_g[n] = 0; cl.free_c[n] -= cs2; cl.free_m[n] -= ms2; cl.owner[n] = j;
                if (first < 0) first = n;
                ++taken;
            }
    }
    V.cls[j] = kind == PIECES ? new_cls : -1;
    ha.node = first;
    ha.packed = pack(gi2, ci2, -1, false, pk_fz_g(ha.packed), pk_fz_c(ha.packed));
    hb.val = v; hb.plan = plan; hb.f_level = f;
    return true;
}

__global__ void __launch_bounds__(ROUND_THREADS, 1)
greedy_round_spread_kernel(const __grid_constant__ Space sp, const __grid_constant__ SpreadArgs S,
                           const rubick_job *__restrict__ jobs, int J,
                           const float *__restrict__ cv, const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                           const uint32_t *__restrict__ feas, int N, int max_steps, rubick_assignment *__restrict__ out,
                           rubick_node *__restrict__ node_out, int32_t *__restrict__ step_log, HotA *hotA, HotB *hotB,
                           int32_t *pieces, int32_t *cls_out, uint32_t *__restrict__ status, int32_t *__restrict__ steps_out)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ RoundShared sh;
    __shared__ int s_ok;

    // shared layout: free_m [N] i64 | free_g [N] | free_c [N] | owner [N] | ff [n_small * nC] | sf [nK * n_small * nC] bytes
    Cluster cl;
    cl.N = N;
    cl.free_m = reinterpret_cast<int64_t *>(smem_raw);
    cl.free_g = reinterpret_cast<int32_t *>(cl.free_m + N);
    cl.free_c = cl.free_g + N;
    cl.owner = cl.free_c + N;
    cl.ff = cl.owner + N;
    const int n_ff = sp.n_small * sp.nC;
    uint8_t *sf = reinterpret_cast<uint8_t *>(cl.ff + n_ff);
    SpreadView V; V.pieces = pieces; V.cls = cls_out; V.sf = sf;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mt = sp.nM - 1;

    for (int n = tid; n < N; n += ROUND_THREADS) {
        cl.free_g[n] = sp.Gn; cl.free_c[n] = sp.Cn; cl.free_m[n] = sp.Mn; cl.owner[n] = -1;
    }
    for (int j = tid; j < J; j += ROUND_THREADS) {
        const rubick_job *jb = jobs + j;
        const int c0 = min(max(jb->cmin_idx, 0), sp.nC - 1);
        HotA a; a.gain_g = 0.0f; a.gain_c = 0.0f; a.node = -1;
        a.packed = pack(-1, c0, -1, jb->gmin_idx >= 0, false, false);
        HotB b; b.val = 0.0f; b.plan = -1; b.f_level = -1; b.w = jb->w;
        hotA[j] = a; hotB[j] = b;
        cls_out[j] = -1;
    }
    for (size_t i = tid; i < size_t(J) * RUBICK_MAX_PIECES; i += ROUND_THREADS) pieces[i] = -1;
    if (tid == 0) { sh.steps = 0; sh.capped = 0; sh.n_empty = N; }
    __syncthreads();

    // per-step tables: first fit per (GPU level, core level), empty nodes, and per spread class whether enough
    // free pieces exist for (GPU level, core level); one warp per entry
    auto build_tables = [&]() {
        const int n_sf = S.nK * n_ff;
        for (int e = warp; e <= n_ff + n_sf; e += ROUND_WARPS) {
            if (e == n_ff + n_sf) {
                int cnt = 0;
                for (int nb = 0; nb < N; nb += 32) {
                    const int n = nb + lane;
                    cnt += __popc(__ballot_sync(0xffffffffu, n < N && cl.free_g[n] == sp.Gn));
                }
                if (lane == 0) sh.n_empty = cnt;
            } else if (e < n_ff) {
                const int gi = e / sp.nC, ci = e - gi * sp.nC;
                const int n = first_fit_warp(cl, sp.g_levels[gi], sp.c_levels[ci], lane);
                if (lane == 0) cl.ff[e] = n;
            } else {
                const int k = (e - n_ff) / n_ff, r = (e - n_ff) - k * n_ff;
                const int gi = r / sp.nC, ci = r - gi * sp.nC;
                const int a = S.align[k], g2 = sp.g_levels[gi], c2 = sp.c_levels[ci];
                int have = 0;
                if (a > 0 && g2 % a == 0 && g2 > a) {
                    const int cpp = int(cdiv_i64(int64_t(c2) * a, g2));
                    for (int n = lane; n < N; n += 32) have += min(cl.free_g[n] / a, cl.free_c[n] / cpp);
                    have = __reduce_add_sync(0xffffffffu, have);
                    have = have >= g2 / a;
                }
                if (lane == 0) sf[e - n_ff] = uint8_t(have);
            }
        }
    };

    // commit of job j to (gi2, ci2): whole on a node (or on whole nodes) through the plain round's commit when that
    // placement exists and the job does not sit in pieces, otherwise through commit_pieces (one thread)
    auto commit_any = [&](int j, HotA &a, HotB &b, int gi2, int ci2, bool need_gain) -> bool {
        const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
        const bool in_pieces = gi >= 0 && cls_out[j] >= 0;
        if (!in_pieces && placeable(sp, cl, sh.n_empty, gi, ci, a.node, gi2, ci2))
            return commit_warp(sp, cl, sh.n_empty, cv, cp, cg, feas, j, a, b, gi2, ci2, need_gain, lane);
        if (lane == 0) {
            HotA a2 = a; HotB b2 = b;
            const bool ok = commit_pieces(sp, cl, S, V, sh.n_empty, cv, cp, cg, feas, j, a2, b2, gi2, ci2, need_gain);
            s_ok = ok ? 1 : 0;
            if (ok) { hotA[j] = a2; hotB[j] = b2; }
        }
        __syncwarp();
        const bool ok = s_ok != 0;
        if (ok) { a = hotA[j]; b = hotB[j]; }
        __syncwarp();
        return ok;
    };

    // ---- Phase A: guaranteed minima, in job order (warp 0; the tables are rebuilt after every placement) ------
    for (int base = 0; base < J; base += 32) {
        const int jj = base + lane;
        const bool want = jj < J && pk_pending(hotA[jj].packed);
        unsigned todo = __ballot_sync(0xffffffffu, want);       // the same in every warp
        while (todo) {
            const int j = base + __ffs(todo) - 1;
            todo &= todo - 1;
            build_tables();
            __syncthreads();
            if (warp == 0) {
                const rubick_job *jb = jobs + j;
                const int gmin = jb->gmin_idx, cmin = max(jb->cmin_idx, 0);
                bool go = gmin < sp.nG && cmin < sp.nC;
                int gi = -1;
                if (go) {
                    const size_t o = curve_idx(sp, j, gmin, cmin, mt);
                    go = __ldg(cp + o) >= 0;
                    // the curve may reach this value with fewer GPUs than the level offers
                    if (go) { gi = level_of_g(sp, __ldg(cg + o)); go = gi >= 0; }
                }
                if (go) {
                    HotA a = hotA[j]; HotB b = hotB[j];
                    if (commit_any(j, a, b, gi, cmin, false) && lane == 0) { hotA[j] = a; hotB[j] = b; }
                }
            }
            __syncthreads();
        }
    }
    __syncthreads();

    // initial gains of every job that may still grow (a job in pieces reads its own class's curves)
    for (int j = tid; j < J; j += ROUND_THREADS) {
        HotA a = hotA[j];
        if (pk_pending(a.packed)) continue;
        const int k = pk_gi(a.packed) >= 0 ? cls_out[j] : -1;
        const Gains r = job_gains(sp, k >= 0 ? S.cv[k] : cv, j, hotB[j].w, pk_gi(a.packed), pk_ci(a.packed), hotB[j].val);
        a.gain_g = r.gain_g; a.gain_c = r.gain_c;
        a.packed = pack(pk_gi(a.packed), pk_ci(a.packed), r.next_g, false, false, false);
        hotA[j] = a;
    }
    __syncthreads();

    // ---- Phase B: greedy increments -----------------------------------------------------------------
    for (;;) {
        build_tables();
        __syncthreads();
        const int n_empty = sh.n_empty;
        unsigned long long best_g = 0ull, best_c = 0ull;
        for (int j = tid; j < J; j += ROUND_THREADS) {
            const HotA a = hotA[j];
            const unsigned long long kg = (static_cast<unsigned long long>(__float_as_uint(a.gain_g)) << 32) | (0xffffffffu - uint32_t(j));
            const unsigned long long kc = (static_cast<unsigned long long>(__float_as_uint(a.gain_c)) << 32) | (0xffffffffu - uint32_t(j));
            const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
            if (a.gain_g > 0.0f && kg > best_g && placeable_spread(sp, cl, S, V, n_empty, j, gi, ci, a.node, pk_next_gi(a.packed), ci)) best_g = kg;
            if (a.gain_c > 0.0f && kc > best_c && placeable_spread(sp, cl, S, V, n_empty, j, gi, ci, a.node, gi, ci + 1)) best_c = kc;
        }
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
            if (sel_j >= 0) {
                const int j = sel_j;
                HotA a = hotA[j]; HotB b = hotB[j];
                const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
                const int gi2 = sel_type == 0 ? pk_next_gi(a.packed) : gi;
                const int ci2 = sel_type == 0 ? ci : ci + 1;
                const bool ok = commit_any(j, a, b, gi2, ci2, true);
                bool fz_g = pk_fz_g(a.packed), fz_c = pk_fz_c(a.packed);
                if (!ok) { if (sel_type == 0) fz_g = true; else fz_c = true; }
                const int k = pk_gi(a.packed) >= 0 ? cls_out[j] : -1;
                const Gains r = job_gains(sp, k >= 0 ? S.cv[k] : cv, j, b.w, pk_gi(a.packed), pk_ci(a.packed), b.val);
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
            if (cls_out[j] >= 0) {
                int np = 0;
                while (np < RUBICK_MAX_PIECES && pieces[size_t(j) * RUBICK_MAX_PIECES + np] >= 0) ++np;
                r.n_nodes = np;
            }
            r.thr = b.val; r.status = RUBICK_RUNNING; r.m_level = b.f_level;
        } else {
            r.g = 0; r.c = 0; r.m_bytes = 0; r.plan = -1; r.first_node = -1; r.n_nodes = 0; r.thr = 0.0f;
            r.status = pk_pending(a.packed) ? RUBICK_PENDING : RUBICK_UNALLOCATED; r.m_level = -1;
            cls_out[j] = -1;
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

}  // namespace rubick

using namespace rubick;

extern "C" int rubick_greedy_round_spread(rubick_ctx *ctx, const rubick_job *d_jobs, int J,
                                          const float *d_curve_val, const int32_t *d_curve_plan, const int32_t *d_curve_g,
                                          const uint32_t *d_feas, const rubick_spread_class *h_classes, int n_classes,
                                          const rubick_cluster *h_cluster, int max_steps, rubick_assignment *d_out,
                                          rubick_node *d_node_out, int32_t *d_step_log, int32_t *d_pieces, int32_t *d_class,
                                          int32_t *h_steps)
{
    if (!ctx) return RUBICK_EINVAL;
    if (!ctx->has_space) return fail(ctx, RUBICK_ESTATE, "no plan space: call rubick_set_space first");
    if (J < 0 || max_steps < 0) return fail(ctx, RUBICK_EINVAL, "negative job count or max_steps");
    if (J >= (1 << 29)) return fail(ctx, RUBICK_EINVAL, "too many jobs");
    if (!h_cluster || h_cluster->n_nodes < 1 || h_cluster->n_nodes > RUBICK_MAX_NODES) return fail(ctx, RUBICK_EINVAL, "cluster: 1 .. RUBICK_MAX_NODES nodes");
    if (h_cluster->n_tenants != 0) return fail(ctx, RUBICK_EINVAL, "rubick_greedy_round_spread: tenant quotas are not supported (n_tenants must be 0)");
    if (n_classes < 0 || n_classes > RUBICK_MAX_SPREAD_CLASSES || (n_classes > 0 && !h_classes)) return fail(ctx, RUBICK_EINVAL, "0 .. RUBICK_MAX_SPREAD_CLASSES spread classes");
    if (ctx->space.Gn > RUBICK_MAX_PIECES) return fail(ctx, RUBICK_EINVAL, "spread placement: at most 32 GPUs per node");
    if (J > 0 && (!d_jobs || !d_curve_val || !d_curve_plan || !d_curve_g || !d_feas || !d_out || !d_pieces || !d_class)) return fail(ctx, RUBICK_EINVAL, "null pointer");
    SpreadArgs S;
    S.nK = n_classes;
    for (int k = 0; k < RUBICK_MAX_SPREAD_CLASSES; ++k) { S.align[k] = 0; S.cv[k] = nullptr; S.cp[k] = nullptr; S.cg[k] = nullptr; S.feas[k] = nullptr; }
    for (int k = 0; k < n_classes; ++k) {
        const rubick_spread_class &c = h_classes[k];
        if (c.align < 1 || c.align >= ctx->space.Gn || (c.align & (c.align - 1))) return fail(ctx, RUBICK_EINVAL, "spread class: align must be a power of two below gpus_per_node");
        if (J > 0 && (!c.d_curve_val || !c.d_curve_plan || !c.d_curve_g || !c.d_feas)) return fail(ctx, RUBICK_EINVAL, "spread class: null table");
        S.align[k] = c.align; S.cv[k] = c.d_curve_val; S.cp[k] = c.d_curve_plan; S.cg[k] = c.d_curve_g; S.feas[k] = c.d_feas;
    }
    const Space &sp = ctx->space;
    const int N = h_cluster->n_nodes;
    const size_t n_ff = size_t(sp.n_small) * sp.nC;
    size_t smem = size_t(N) * 20 + n_ff * 4 + size_t(n_classes) * n_ff;
    smem = (smem + 15) & ~size_t(15);
    if (smem > 200 * 1024) return fail(ctx, RUBICK_EINVAL, "cluster state does not fit shared memory");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaSetDevice");
    const size_t need = size_t(J > 0 ? J : 1) * (sizeof(HotA) + sizeof(HotB));
    if (need > ctx->round_scratch_bytes) {
        if (ctx->d_round_scratch) { cudaStreamSynchronize(ctx->stream); cudaFree(ctx->d_round_scratch); ctx->d_round_scratch = nullptr; ctx->round_scratch_bytes = 0; }
        e = cudaMalloc(&ctx->d_round_scratch, need);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMalloc (round scratch)");
        ctx->round_scratch_bytes = need;
    }
    HotA *ha = reinterpret_cast<HotA *>(ctx->d_round_scratch);
    HotB *hb = reinterpret_cast<HotB *>(reinterpret_cast<unsigned char *>(ctx->d_round_scratch) + size_t(J > 0 ? J : 1) * sizeof(HotA));
    const long long natural = (long long)J * (sp.nG + sp.nC + 2) + 1;
    if ((long long)max_steps > natural) max_steps = int(natural < 0x7fffffffLL ? natural : 0x7fffffffLL);
    e = cudaFuncSetAttribute(greedy_round_spread_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute");
    greedy_round_spread_kernel<<<1, ROUND_THREADS, smem, ctx->stream>>>(sp, S, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas, N,
                                                                        max_steps, d_out, d_node_out, d_step_log, ha, hb, d_pieces, d_class,
                                                                        ctx->d_status, ctx->d_steps);
    count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch greedy_round_spread");
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
