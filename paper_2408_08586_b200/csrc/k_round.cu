// Greedy scheduling round, fast path (paper Section 5.2, Algorithm 1 in marginal-gain form).
//
// Same decisions, step for step, as the plain round in k_sched.cu (largest placeable positive
// GPU gain first, CPU gain when no GPU increment is left, lowest job index on ties, commit with
// the best plan and its host memory), organised so that one step costs a fraction of a microsecond:
//
//   prepare  (grid)   one CTA per job.  Per (job, GPU level, CPU level): the curve entry at the top host-memory
//                     level together with the first feasible memory level of its plan, 16 bytes.  A commit
//                     whose node offers at least that level needs no further table look-up, because
//                     the curve at any level >= the plan's first level equals the curve at the top.
//                     Then, from those values (kept in shared memory), a 32-byte transition record: the gains
//                     a job has once it holds that allocation with the curve's value, the level its GPU gain
//                     refers to and what its two candidates need in order to be placeable.  A batched
//                     increment reads one record instead of a column of the curve.
//   keys     (grid)   every best-effort job starts unallocated, and its first increment (smallest
//                     GPU level with a non-zero curve at its starting CPU level) and gain are fixed
//                     until it is allocated: one 64-bit key (class = target levels | gain | ~job).
//                     Guaranteed jobs get their Phase-A target resolved here too.
//   sort     (grid)   bitonic sort of the keys, tiles in shared memory; up to eight tiles in one launch by a
//                     thread-block cluster (wide strides through the partner CTA's shared memory), more with wide
//                     strides in global memory: inside a class (same target levels = same placement test) only the
//                     first unconsumed job can ever be selected.
//   round    (1 CTA)  persistent loop.  Shared memory holds one word per node (free GPUs << 16 | free
//                     cores), free memory and whole-node owners, the table "most free cores among nodes
//                     with >= g free GPUs" (a job of g GPUs and c cores fits some node exactly when that
//                     entry is >= c), the head of every class, one 36-byte slot per RUNNING job (scan state
//                     + what its two candidates need to be placeable) and a bitmap of the nodes the last
//                     iteration changed.  Every scanning warp leaves its four best candidates, the largest key
//                     among the rest and the largest key among the increments that have a gain but no place in
//                     shared memory (the last warp: the best class head and the runner-up key) and looks again
//                     only when one of its slots, a node under them, that table or the number of empty nodes
//                     changed.  Warp 0 holds two offered candidates per lane, picks (type | gain, lowest job)
//                     across them with warp reduce instructions and commits, in the exact order of the
//                     one-step-at-a-time rule, as many steps as it can prove to come next:
//                       - a run of class heads that are rejected (a rejection changes nothing but the head
//                         of its class; every lane settles four entries of the class's sorted list);
//                       - a batch of increments that stay on their own nodes (every lane works out the commits
//                         of its two candidates; the candidates above one threshold - every runner-up,
//                         every candidate that could not be worked out or shares a node with a better one,
//                         every new candidate of the jobs taken - are a prefix of the sequential order
//                         and are committed together);
//                       - otherwise a chain of general commits (migrations, growth onto whole nodes, class heads
//                         that succeed): the offered candidates and the first entries of the best class, staged
//                         in the rule's order, are committed one after another on the real cluster state while
//                         the next key exceeds every key not offered, every new candidate of the jobs committed
//                         before it and, once resources were given back, every increment that had no place.
//
// All gain arithmetic uses __fmul_rn / __fsub_rn / __fdiv_rn (one rounding per operation, never
// fused) so that decisions are reproducible bit for bit.  Every loop is bounded (steps by
// max_steps, scans by the node / level counts); nothing spins on memory.

#include "rubick_internal.cuh"
#include <cooperative_groups.h>

namespace rubick {
namespace fastround {

constexpr int RT = 512;                 // threads of the persistent round kernel
constexpr int RW = RT / 32;
constexpr size_t SMEM_LIMIT = 200 * 1024;
constexpr int RUN_U = 4;                // a run of failing class heads settles up to 32 * RUN_U entries a turn

typedef unsigned long long u64;

struct HotCurve { float val; int32_t plan; int32_t f; int32_t ok; };                        // 16 bytes
struct PhaseA { int32_t gi, ci; float val; int32_t plan; int32_t f; int32_t ok; float w; int32_t pad; };   // 32 bytes
struct SlotA { float gain_g, gain_c; uint32_t packed; int32_t node; };
struct SlotB { float val; int32_t plan; int32_t f_level; float w; };

// sort key of an unallocated job: [63:53] class = gi2 * 64 + ci | [52:21] gain bits | [20:0] ~job
constexpr int KEY_JOB_BITS = 21;
constexpr u64 KEY_JOB_MASK = (1ull << KEY_JOB_BITS) - 1;
__device__ __forceinline__ int key_job(u64 k) { return int(KEY_JOB_MASK - (k & KEY_JOB_MASK)); }
__device__ __forceinline__ uint32_t key_gain_bits(u64 k) { return uint32_t(k >> KEY_JOB_BITS); }
__device__ __forceinline__ int key_class(u64 k) { return int(k >> 53); }

// selection key of a step (32 bits): [31] 1 = GPU increment | [30:0] bits of the positive gain;
// equal keys go to the lowest job index

// slot.packed: [5:0] g level | [12:6] c level | [18:13] target g level + 1 | [20] GPU frozen | [21] CPU frozen
__device__ __forceinline__ uint32_t pack(int gi, int ci, int next_gi, bool fz_g, bool fz_c)
{
    return uint32_t(gi) | (uint32_t(ci) << 6) | (uint32_t(next_gi + 1) << 13) | (uint32_t(fz_g) << 20) | (uint32_t(fz_c) << 21);
}
__device__ __forceinline__ int pk_gi(uint32_t p) { return int(p & 63u); }
__device__ __forceinline__ int pk_ci(uint32_t p) { return int((p >> 6) & 127u); }
__device__ __forceinline__ int pk_next_gi(uint32_t p) { return int((p >> 13) & 63u) - 1; }
__device__ __forceinline__ bool pk_fz_g(uint32_t p) { return (p >> 20) & 1u; }
__device__ __forceinline__ bool pk_fz_c(uint32_t p) { return (p >> 21) & 1u; }

__device__ __forceinline__ size_t curve_idx(const Space &sp, int j, int gi, int ci, int mi)
{
    return ((size_t(j) * sp.nG + gi) * sp.nC + ci) * sp.nM + mi;
}
__device__ __forceinline__ size_t hc_idx(const Space &sp, int j, int gi, int ci) { return (size_t(j) * sp.nG + gi) * sp.nC + ci; }
__device__ __forceinline__ int64_t cdiv64(int64_t a, int64_t b) { return (a + b - 1) / b; }
// ceil(a / k), a >= 0, k >= 1: node counts of jobs on whole nodes usually are powers of two (a shift, no division)
__device__ __forceinline__ int cdiv_k(int a, int k) { return (k & (k - 1)) ? (a + k - 1) / k : (a + k - 1) >> (__ffs(k) - 1); }
__device__ __forceinline__ int64_t cdiv64_k(int64_t a, int k) { return (k & (k - 1)) ? (a + k - 1) / k : (a + k - 1) >> (__ffs(k) - 1); }
__device__ __forceinline__ HotCurve load_hc(const HotCurve *p)
{
    const int4 v = *reinterpret_cast<const int4 *>(p);
    HotCurve h; h.val = __int_as_float(v.x); h.plan = v.y; h.f = v.z; h.ok = v.w;
    return h;
}

// Requests the curve entry and the transition record of (j, gi, ci) into the L1 cache: the job that was just committed
// may offer this allocation as its next candidate, and the turn that works the candidate out then finds them near.
__device__ __forceinline__ void prefetch_target(const Space &sp, const HotCurve *hc, const void *tr32, int j, int gi, int ci)
{
    const size_t o = hc_idx(sp, j, gi, ci);
    asm volatile("prefetch.global.L1 [%0];" :: "l"(hc + o));
    asm volatile("prefetch.global.L1 [%0];" :: "l"(static_cast<const char *>(tr32) + o * 32));
}

// ---- keys: first increment of every best-effort job, Phase-A target of every guaranteed job -------
__global__ void round_keys_kernel(const __grid_constant__ Space sp, const rubick_job *__restrict__ jobs, int J,
                                  const HotCurve *__restrict__ hc, const int32_t *__restrict__ cp,
                                  const int32_t *__restrict__ cg, u64 *__restrict__ keys, int n_pad,
                                  PhaseA *__restrict__ pa, rubick_assignment *__restrict__ out,
                                  int32_t *__restrict__ is_guar)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n_pad) return;
    u64 key = 0ull;
    if (j < J) {
        const rubick_job *jb = jobs + j;
        const int gmin = jb->gmin_idx;
        const float w = jb->w;
        PhaseA a; a.gi = -2; a.ci = 0; a.val = 0.0f; a.plan = -1; a.f = -1; a.ok = 0; a.w = w; a.pad = jb->tenant;
        if (gmin < 0) {
            const int ci = min(max(jb->cmin_idx, 0), sp.nC - 1);
            for (int gi = 0; gi < sp.nG; ++gi) {
                const float v = hc[hc_idx(sp, j, gi, ci)].val;
                if (v > 0.0f) {
                    const float gain = __fdiv_rn(__fsub_rn(__fmul_rn(w, v), 0.0f), float(sp.g_levels[gi]));
                    if (gain > 0.0f)
                        key = (u64(gi * 64 + ci) << 53) | (u64(__float_as_uint(gain)) << KEY_JOB_BITS) | (KEY_JOB_MASK - u64(j));
                    break;
                }
            }
        } else {
            // guaranteed: placed in Phase A at (gmin, cmin) with the GPU count the curve really uses
            a.gi = -1;
            const int cmin = max(jb->cmin_idx, 0);
            if (gmin < sp.nG && cmin < sp.nC) {
                const size_t o = curve_idx(sp, j, gmin, cmin, sp.nM - 1);
                if (__ldg(cp + o) >= 0) {
                    // the curve may reach this value with fewer GPUs than the level offers
                    const int gu = __ldg(cg + o);
                    int gi = -1;
                    for (int i = 0; i < sp.nG; ++i) if (sp.g_levels[i] == gu) gi = i;
                    if (gi >= 0) {
                        const HotCurve h = load_hc(hc + hc_idx(sp, j, gi, cmin));
                        a.gi = gi; a.ci = cmin; a.val = h.val; a.plan = h.plan; a.f = h.f; a.ok = h.ok;
                    }
                }
            }
        }
        reinterpret_cast<int4 *>(pa + j)[0] = make_int4(a.gi, a.ci, __float_as_int(a.val), a.plan);
        reinterpret_cast<int4 *>(pa + j)[1] = make_int4(a.f, a.ok, __float_as_int(a.w), a.pad);      // pad carries the tenant
        // the result every job has until the round places it, and the mark the round builds its Phase-A list from
        rubick_assignment r;
        r.g = 0; r.c = 0; r.m_bytes = 0; r.plan = -1; r.first_node = -1; r.n_nodes = 0; r.thr = 0.0f;
        r.status = a.gi != -2 ? RUBICK_PENDING : RUBICK_UNALLOCATED; r.m_level = -1;
        out[j] = r;
        is_guar[j] = a.gi != -2;
    }
    keys[j] = key;
}

// ---- sort: descending bitonic sort of n (power of two) keys, then the weights in sorted order -----
// Tiles of SORT_TILE keys live in shared memory, one CTA each: the stages up to the tile size run entirely there,
// a later stage k does its passes with strides of a tile or more in global memory (one small launch each) and
// the remaining ones in shared memory again.
constexpr int SORT_TILE = 2048;
constexpr int SORT_T = SORT_TILE / 2;   // one thread per compare-exchange pair of a tile

__device__ __forceinline__ void sort_pair(u64 *a, int i, int p, bool desc)
{
    const u64 x = a[i], y = a[p];
    if (desc ? (x < y) : (x > y)) { a[i] = y; a[p] = x; }
}

// stages k_from .. k_to of the tile starting at blockIdx.x * tile: for every stage the passes with stride
// min(k / 2, tile / 2) down to 1.  last: also writes the weights in sorted order.
__global__ void __launch_bounds__(SORT_T)
round_sort_tile_kernel(u64 *__restrict__ keys, int n, int tile, int k_from, int k_to, int last,
                       const rubick_job *__restrict__ jobs, float *__restrict__ sorted_w)
{
    __shared__ u64 a[SORT_TILE];
    const int base = blockIdx.x * tile;
    for (int i = threadIdx.x; i < tile; i += SORT_T) a[i] = keys[base + i];
    __syncthreads();
    for (int k = k_from; k <= k_to; k <<= 1)
        for (int s = min(k >> 1, tile >> 1); s > 0; s >>= 1) {
            for (int t = threadIdx.x; t < (tile >> 1); t += SORT_T) {
                const int i = ((t & ~(s - 1)) << 1) | (t & (s - 1));
                sort_pair(a, i, i | s, ((base + i) & k) == 0);
            }
            __syncthreads();
        }
    for (int i = threadIdx.x; i < tile; i += SORT_T) {
        const u64 k = a[i];
        keys[base + i] = k;
        if (last) sorted_w[base + i] = k ? jobs[key_job(k)].w : 0.0f;
    }
}

// The whole sort in one launch when the keys fit the shared memory of one thread-block cluster (up to eight tiles): a
// pass with a stride of a tile or more pairs every key with one in another CTA's shared memory, which the CTA reads and
// writes directly; each of the two CTAs settles half of the pairs they share.  Every CTA runs the same passes, so the
// cluster barriers match; the last pass that touches another CTA's memory is followed by one.
__global__ void __launch_bounds__(SORT_T)
round_sort_cluster_kernel(u64 *__restrict__ keys, int n, const rubick_job *__restrict__ jobs, float *__restrict__ sorted_w)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ u64 a[SORT_TILE];
    const int rank = int(cluster.block_rank());
    const int base = rank * SORT_TILE;
    for (int i = threadIdx.x; i < SORT_TILE; i += SORT_T) a[i] = keys[base + i];
    __syncthreads();
    for (int k = 2; k <= n; k <<= 1) {
        for (int s = k >> 1; s >= SORT_TILE; s >>= 1) {
            cluster.sync();                                  // every CTA is through with the step before
            const int bit = s / SORT_TILE;
            const int other = rank ^ bit;
            const bool low = (rank & bit) == 0;              // this CTA holds the lower key of every pair it shares with `other`
            u64 *b = cluster.map_shared_rank(a, other);
            const int li = threadIdx.x + (low ? 0 : SORT_T); // the lower tile settles the first half of the indices
            const int lo_index = (low ? base : other * SORT_TILE) + li;
            u64 *lo = low ? a : b, *hi = low ? b : a;
            const u64 x = lo[li], y = hi[li];
            if (((lo_index & k) == 0) ? (x < y) : (x > y)) { lo[li] = y; hi[li] = x; }
        }
        if (k > SORT_TILE) cluster.sync(); else __syncthreads();
        for (int s = min(k >> 1, SORT_TILE >> 1); s > 0; s >>= 1) {
            const int t = threadIdx.x;
            const int i = ((t & ~(s - 1)) << 1) | (t & (s - 1));
            sort_pair(a, i, i | s, ((base + i) & k) == 0);
            __syncthreads();
        }
    }
    for (int i = threadIdx.x; i < SORT_TILE; i += SORT_T) {
        const u64 k = a[i];
        keys[base + i] = k;
        sorted_w[base + i] = k ? jobs[key_job(k)].w : 0.0f;
    }
}
constexpr int SORT_CLUSTER_MAX = 8;         // tiles one launch can sort (the portable cluster size)

// one pass of stage k with stride s (a tile or more) in global memory; one thread per pair
__global__ void round_sort_pass_kernel(u64 *__restrict__ keys, int n, int k, int s)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (n >> 1)) return;
    const int i = ((t & ~(s - 1)) << 1) | (t & (s - 1));
    sort_pair(keys, i, i | s, (i & k) == 0);
}

// ---- the persistent round ---------------------------------------------------------------------------

// what a slot's two candidates need in order to be placeable, precomputed when its gains are
struct SlotC {
    uint8_t gkind, ckind;     // K_SINGLE / K_MULTI_WHOLE / K_MULTI_PART / K_NONE
    uint8_t gidx, cidx;       // GPU level whose "most free cores" entry decides a migration
    int16_t dg, need, dc;     // extra GPUs on the own node / empty nodes needed / extra cores on the own node
    int16_t c, c2, g;         // cores held, cores wanted, GPUs held
};
enum : uint8_t { K_SINGLE = 0, K_MULTI_WHOLE = 1, K_MULTI_PART = 2, K_NONE = 3 };

constexpr int SCAN_WARPS = RW - 1;          // all warps but the last scan running jobs, the last one the class heads
constexpr int SCAN_T = SCAN_WARPS * 32;
constexpr int OFFER = 4;                    // candidates every scanning warp offers
constexpr int N_GROUPS = OFFER * SCAN_WARPS + 1;   // candidates seen by warp 0: the best OFFER of every scanning warp + the best class head
constexpr int CLS_G = N_GROUPS - 1;
constexpr int N_CAND = 64;                  // warp 0 holds two candidates per lane: lane l those of index l and l + 32
static_assert(N_GROUPS <= N_CAND, "warp 0 holds two candidates per lane");
// the flag that makes the warp owning slot s look again (flags sit at the index of the warp's first candidate)
__device__ __forceinline__ int dirty_of(int s) { return ((s % SCAN_T) >> 5) * OFFER; }

// node n: gc[n] = free GPUs << 16 | free cores (padding entries are 0: they never fit anything)
__device__ __forceinline__ int fg_of(int w) { return w >> 16; }
__device__ __forceinline__ int fc_of(int w) { return w & 0xffff; }

struct Views {
    int64_t *free_m;
    int32_t *gc, *owner;
    int32_t *maxc;                // [n_small] most free cores among nodes with at least g_levels[i] free GPUs, -1 if none
    int32_t *cls_ptr, *cls_end; u64 *cls_top; float *cls_w;
    int32_t *ccls;                // compact list of the non-empty classes: dense index | gi2 << 16 | ci2 << 24
    SlotA *sa; SlotB *sb; SlotC *sc; int32_t *sj;
    const int32_t *gl, *clv;      // GPU / CPU level values in shared memory (lanes index them divergently)
    const int64_t *ml;            // memory level values, likewise
    uint32_t *tb;                 // bit n set: the last iteration changed the free GPUs / cores of node n
    int N, N_pad;
};

struct Shared {
    uint32_t red_key[N_CAND]; int32_t red_j[N_CAND]; uint32_t red_pay[N_CAND];   // the offered candidates; they stay until their warp looks again
    uint32_t red_key2[N_CAND];    // at a warp's first index: largest key it did not offer (keys only: ties are resolved conservatively);
                                  // at the next: largest key among the increments it found without a place
    int dirty[N_CAND];            // (at a warp's first index) must look again: one of its slots (or a class head) changed
    int n_empty, n_slots, steps, capped, stop, n_guar, n_ccls;
    int ver;                      // bumped whenever maxc[] or the empty-node count changes
    int maxc_dirty;               // the last commit may have changed maxc[]
    int batch_go;                 // this turn is a batch of increments: warp 1 works out half of the candidates
    unsigned acc_b; int steps0_b; int order_b[32];   // ... and, of its half, which are taken, the step count before them, their places in the step log
    int scan_cnt[RW];
    int empty_lo;                 // no node below this index is empty (whole multiples of 32 after a search)
    int4 pa_rec[32][2]; int pa_job[32];   // Phase A: the records of the 32 jobs being worked on
    int pa_commits;               // Phase A: jobs placed so far
    int ff_pos[RUBICK_MAX_G_LEVELS];   // Phase A: no node below this index has g_levels[i] free GPUs
    alignas(16) unsigned long long sel[N_CAND];   // batch selection: one ordering word per candidate (read two at a time)
};

// warp-cooperative: first node with at least g free GPUs and c free cores, -1 if none
__device__ int first_fit_warp(const Views &v, int g, int c, int lane)
{
    const int4 *w4 = reinterpret_cast<const int4 *>(v.gc);
    for (int base = 0; base < v.N_pad; base += 128) {
        const int4 x = w4[(base >> 2) + lane];
        int first = -1;
        if (fg_of(x.w) >= g && fc_of(x.w) >= c) first = 3;
        if (fg_of(x.z) >= g && fc_of(x.z) >= c) first = 2;
        if (fg_of(x.y) >= g && fc_of(x.y) >= c) first = 1;
        if (fg_of(x.x) >= g && fc_of(x.x) >= c) first = 0;
        const unsigned b = __ballot_sync(0xffffffffu, first >= 0);
        if (b) return __shfl_sync(0xffffffffu, base + 4 * lane + first, __ffs(b) - 1);
    }
    return -1;
}

// The same while free GPUs only shrink (Phase A): ff_pos[gi] is a node index below which no node has g free
// GPUs any more, so the search starts there, 32 nodes at a time, and moves the mark up to the first node that
// still has them.
__device__ int first_fit_from_mark(const Views &v, Shared &sh, int gi, int g, int c, int lane)
{
    const int need = (g << 16) | c;          // a word fits when it is at least `need` and its core field at least c
    int first_g = -1, found = -1;
    for (int pos = sh.ff_pos[gi]; pos < v.N && found < 0; pos += 32) {
        const int n = pos + lane;
        const int w = n < v.N_pad ? v.gc[n] : 0;
        const unsigned bg = __ballot_sync(0xffffffffu, w >= (g << 16));
        const unsigned bf = __ballot_sync(0xffffffffu, w >= need && fc_of(w) >= c);
        if (first_g < 0 && bg) first_g = pos + __ffs(bg) - 1;
        if (bf) found = pos + __ffs(bf) - 1;
    }
    sh.ff_pos[gi] = first_g >= 0 ? first_g : v.N;       // the same value from every lane: each sees its own store afterwards
    return found;
}

// warp-cooperative: maxc[] for every level in one sweep over the node words (lane 0 stores).  Levels ascend, so
// a node counts for the levels below the first one it has too few free GPUs for.
__device__ void rebuild_maxc_warp(const Space &sp, const Views &v, int lane)
{
    const int4 *w4 = reinterpret_cast<const int4 *>(v.gc);
    for (int i0 = 0; i0 < sp.n_small; i0 += 4) {
        int g_[4], m_[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { g_[u] = i0 + u < sp.n_small ? v.gl[i0 + u] : 0x7fffffff; m_[u] = -1; }
        for (int base = 0; base < v.N_pad; base += 128) {
            const int4 x = w4[(base >> 2) + lane];
            const int w_[4] = { x.x, x.y, x.z, x.w };
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int u = 0; u < 4; ++u) m_[u] = max(m_[u], fg_of(w_[q]) >= g_[u] ? fc_of(w_[q]) : -1);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int m = __reduce_max_sync(0xffffffffu, m_[u]);
            if (lane == 0 && i0 + u < sp.n_small) v.maxc[i0 + u] = m;
        }
    }
}

// warp-cooperative: most free cores among the nodes with at least g free GPUs (-1 if none).  A job of
// g GPUs and c cores fits some node as a whole exactly when this is >= c.
__device__ int max_cores_warp(const Views &v, int g, int lane)
{
    const int4 *w4 = reinterpret_cast<const int4 *>(v.gc);
    int m = -1;
    for (int base = 0; base < v.N_pad; base += 128) {
        const int4 x = w4[(base >> 2) + lane];
        m = max(m, fg_of(x.x) >= g ? fc_of(x.x) : -1);
        m = max(m, fg_of(x.y) >= g ? fc_of(x.y) : -1);
        m = max(m, fg_of(x.z) >= g ? fc_of(x.z) : -1);
        m = max(m, fg_of(x.w) >= g ? fc_of(x.w) : -1);
    }
    return __reduce_max_sync(0xffffffffu, m);
}

struct Committed { int first; float val; int plan; int f; int freed; };      // after a failure: first = -2 if no job with these target levels could have been placed; freed: the job left a node

// warp-cooperative: rebuilds maxc[] like rebuild_maxc_warp and tells whether an entry changed (same answer on every lane)
__device__ bool rebuild_maxc_changed(const Space &sp, const Views &v, int lane)
{
    const int old = lane < sp.n_small ? v.maxc[lane] : 0;
    __syncwarp();
    rebuild_maxc_warp(sp, v, lane);
    __syncwarp();
    return __any_sync(0xffffffffu, lane < sp.n_small && v.maxc[lane] != old);
}

// How the caller of commit_warp keeps the derived state current:
//   COMMIT_TURN   one commit a turn: sh.maxc_dirty / sh.ver and the bitmap of changed nodes tell the block what changed
//   COMMIT_PHASE_A free resources only shrink: the search starts at the first-fit marks, maxc[] is rebuilt here
//   COMMIT_CHAIN  several commits a turn: maxc[] is rebuilt here, sh.ver and the bitmap as for COMMIT_TURN
enum { COMMIT_TURN = 0, COMMIT_PHASE_A = 1, COMMIT_CHAIN = 2 };

// Commit job j to (gi2, ci2); one warp, all lanes, uniform control flow.  `alloc` (compile time): the job holds
// (gi, ci) on `node` with value val_cur and memory level f_cur.  cand = curve entry of the target at
// the top memory level.  On success node state and empty-node count are current.
template <bool alloc, int mode>
__device__ bool commit_warp(const Space &sp, const Views &v, Shared &sh, const float *__restrict__ cv,
                            const int32_t *__restrict__ cp, const int32_t *__restrict__ cg,
                            const uint32_t *__restrict__ feas, int j, int gi, int ci, int node,
                            float val_cur, int f_cur, int gi2, int ci2, HotCurve cand, bool need_gain,
                            int lane, Committed &out)
{
    // level values from their shared-memory copies (an indexed read of the constant bank takes longer)
    const int g = alloc ? v.gl[gi] : 0, c = alloc ? v.clv[ci] : 0;
    const int64_t m_cur = alloc ? v.ml[f_cur] : 0;
    const int g2 = v.gl[gi2], c2 = v.clv[ci2];
    const int k = alloc ? max(g >> sp.log2Gn, 1) : 0;
    const int n_empty = sh.n_empty;

    int k2 = 1, target = -1, need_new = 0;
    bool stay = false;
    if (g2 <= sp.Gn) {
        if (alloc) { const int w = v.gc[node]; stay = fg_of(w) >= g2 - g && fc_of(w) >= c2 - c; }
        if (stay) target = node;
        else if (v.maxc[gi2] >= c2) target = mode == COMMIT_PHASE_A ? first_fit_from_mark(v, sh, gi2, g2, c2, lane) : first_fit_warp(v, g2, c2, lane);
        if (target < 0) { out.first = -2; return false; }
    } else {
        k2 = g2 >> sp.log2Gn;
        if (cdiv_k(c2, k2) > sp.Cn) return false;
        if (alloc && g >= sp.Gn) { stay = true; need_new = k2 - k; if (n_empty < need_new) return false; }
        else {
            need_new = k2;
            const int empty = n_empty + ((alloc && fg_of(v.gc[node]) + g == sp.Gn) ? 1 : 0);
            if (empty < need_new) return false;
        }
    }

    // highest memory level whose per-node share fits: ceil(m / k2) <= avail  <=>  m <= avail * k2
    const int64_t avail = k2 > 1 ? sp.Mn : v.free_m[target] + ((stay && alloc) ? m_cur : 0);
    const bool fits = lane < sp.nM && v.ml[lane < sp.nM ? lane : 0] <= avail * k2;
    const unsigned fb = __ballot_sync(0xffffffffu, fits);
    if (!fb) { out.first = -2; return false; }      // the node found has too little memory for any level
    const int mi = 31 - __clz(fb);

    float val; int plan, f; bool okg;
    if (cand.plan >= 0 && cand.f >= 0 && cand.f <= mi) {
        // the top-level best plan is feasible at level mi, hence also the best one there
        val = cand.val; plan = cand.plan; f = cand.f; okg = cand.ok != 0;
    } else {
        const size_t o = curve_idx(sp, j, gi2, ci2, mi);
        val = __ldg(cv + o); plan = __ldg(cp + o); okg = __ldg(cg + o) == g2;
        f = -1;
        if (plan >= 0 && plan < sp.P) f = __ffs(__ldg(feas + size_t(j) * sp.P + plan)) - 1;
    }
    if (plan < 0 || plan >= sp.P || !(val > 0.0f) || !okg) return false;
    if (need_gain && alloc && !(val > val_cur)) return false;
    if (f < 0 || f > mi) return false;
    const int64_t m2 = v.ml[f];

    // ---- node bookkeeping ------------------------------------------------------------------------
    int first = -1, d_empty = 0;
    bool maxc_dirty = true;
    int t0 = -1, t1 = -1;
    out.freed = alloc && !stay;
    if (k2 == 1) {
        const int moved = alloc && !stay;
        const int w_old_n = moved ? v.gc[node] : 0, w_old_t = v.gc[target];
        const int w_new_n = w_old_n + (g << 16) + c;
        const int w_new_t = stay ? w_old_t - ((g2 - g) << 16) - (c2 - c) : w_old_t - (g2 << 16) - c2;
        if (lane == 0) {
            if (moved) { v.gc[node] = w_new_n; v.free_m[node] += m_cur; }
            v.gc[target] = w_new_t;
            v.free_m[target] -= stay ? m2 - m_cur : m2;
        }
        if (moved && fg_of(w_new_n) == sp.Gn) { d_empty += 1; if (lane == 0 && node < sh.empty_lo) sh.empty_lo = node; }
        if (!stay && fg_of(w_old_t) == sp.Gn) d_empty -= 1;
        first = target; t1 = target; t0 = moved ? node : -1;
        // can maxc[] have changed?  lane i answers for GPU level i
        bool ch = false;
        if (lane < sp.n_small) {
            const int gl = v.gl[lane], mx = v.maxc[lane];
            const int ot = fg_of(w_old_t) >= gl ? fc_of(w_old_t) : -1, nt = fg_of(w_new_t) >= gl ? fc_of(w_new_t) : -1;
            ch = (ot == mx && nt < ot) || nt > mx;
            if (moved) {
                const int on = fg_of(w_old_n) >= gl ? fc_of(w_old_n) : -1, nn = fg_of(w_new_n) >= gl ? fc_of(w_new_n) : -1;
                ch = ch || (on == mx && nn < on) || nn > mx;
            }
        }
        // while an empty node remains every entry equals the node's core count: nothing to recompute
        if (n_empty + d_empty > 0) ch = lane < sp.n_small && v.maxc[lane] != sp.Cn;
        maxc_dirty = __any_sync(0xffffffffu, ch);
    } else {
        const int cs2 = cdiv_k(c2, k2);
        const int64_t ms2 = cdiv64_k(m2, k2);
        if (stay) {
            // whole nodes already held keep their GPUs; only the core / memory shares change
            const int cs1 = cdiv_k(c, alloc ? k : 1);
            const int64_t ms1 = cdiv64_k(m_cur, alloc ? k : 1);
            if (k == 1) {
                if (lane == 0) { v.gc[node] += c - cs2; v.free_m[node] += m_cur - ms2; v.owner[node] = j; }
            } else {
                // the k nodes of a job usually are node .. node + k - 1 (taken together from an empty stretch)
                const int nn = node + lane;
                const bool mine = lane < k && nn < v.N && v.owner[nn] == j;
                if (__popc(__ballot_sync(0xffffffffu, mine)) == k) {
                    if (mine) { v.gc[nn] += cs1 - cs2; v.free_m[nn] += ms1 - ms2; }
                } else {
                    for (int n = lane; n < v.N; n += 32)
                        if (v.owner[n] == j) { v.gc[n] += cs1 - cs2; v.free_m[n] += ms1 - ms2; }
                }
            }
            first = node;
        } else if (alloc) {
            if (lane == 0) { v.gc[node] += (g << 16) + c; v.free_m[node] += m_cur; }
            __syncwarp();
            if (fg_of(v.gc[node]) == sp.Gn) { d_empty += 1; if (lane == 0 && node < sh.empty_lo) sh.empty_lo = node; }
        }
        __syncwarp();
        int taken = 0, base = sh.empty_lo & ~31;          // every empty node below the search's last look is taken
        for (; base < v.N && taken < need_new; base += 32) {
            const int n = base + lane;
            const bool empty = n < v.N && fg_of(v.gc[n]) == sp.Gn;
            const unsigned b = __ballot_sync(0xffffffffu, empty);
            const int rank = __popc(b & ((1u << lane) - 1u));
            if (empty && taken + rank < need_new) { v.gc[n] -= (sp.Gn << 16) + cs2; v.free_m[n] -= ms2; v.owner[n] = j; }
            if (b) { const int lowest = base + __ffs(b) - 1; if (first < 0 || lowest < first) first = lowest; }
            taken += __popc(b);
        }
        if (lane == 0 && need_new > 0) sh.empty_lo = base - 32;
        d_empty -= need_new;
        // while an empty node remains every entry of maxc[] equals the node's core count: nothing to recompute
        if (n_empty + d_empty > 0) maxc_dirty = __any_sync(0xffffffffu, lane < sp.n_small && v.maxc[lane] != sp.Cn);
    }
    __syncwarp();
    if (mode == COMMIT_PHASE_A) {
        if (maxc_dirty) rebuild_maxc_warp(sp, v, lane);
        if (lane == 0) sh.n_empty = n_empty + d_empty;
        __syncwarp();
    } else if (mode == COMMIT_CHAIN) {
        const bool changed = maxc_dirty && rebuild_maxc_changed(sp, v, lane);
        if (lane == 0) {
            sh.n_empty = n_empty + d_empty;
            if (t0 >= 0) v.tb[t0 >> 5] |= 1u << (t0 & 31);
            if (t1 >= 0) v.tb[t1 >> 5] |= 1u << (t1 & 31);
            if (d_empty != 0 || k2 > 1 || changed) sh.ver += 1;
        }
        __syncwarp();
    } else if (lane == 0) {
        sh.n_empty = n_empty + d_empty;
        sh.maxc_dirty = maxc_dirty;
        if (t0 >= 0) v.tb[t0 >> 5] |= 1u << (t0 & 31);
        if (t1 >= 0) v.tb[t1 >> 5] |= 1u << (t1 & 31);
        if (d_empty != 0 || k2 > 1) sh.ver += 1;
    }
    out.first = first; out.val = val; out.plan = plan; out.f = f;
    return true;
}

// gains of a running job from the values of its curve column (lane i holds the value of GPU level
// gi + 1 + i, vc the value at the next core level); identical on every lane
__device__ __forceinline__ void gains_from_column(const Space &sp, float w, int gi, int ci, float val, float v_lane,
                                                  float vc, int lane, int &next_g, float &gain_g, int &next_c, float &gain_c)
{
    const float vcur = __fmul_rn(w, val);
    const int lvl = gi + 1 + lane;
    const unsigned b = __ballot_sync(0xffffffffu, lvl < sp.nG && v_lane > val);
    next_g = -1; gain_g = 0.0f; next_c = -1; gain_c = 0.0f;
    if (b) {
        const int src = __ffs(b) - 1;
        const float vv = __shfl_sync(0xffffffffu, v_lane, src);
        next_g = gi + 1 + src;
        gain_g = __fdiv_rn(__fsub_rn(__fmul_rn(w, vv), vcur), float(sp.g_levels[next_g] - sp.g_levels[gi]));
    }
    if (ci + 1 < sp.nC) {
        const float gn = __fdiv_rn(__fsub_rn(__fmul_rn(w, vc), vcur), float(sp.c_levels[ci + 1] - sp.c_levels[ci]));
        if (gn > 0.0f) { next_c = ci + 1; gain_c = gn; }
    }
}

// the same for one thread (initial gains of the jobs placed in Phase A)
__device__ void gains_thread(const Space &sp, const HotCurve *__restrict__ hc, int j, float w, int gi, int ci, float val,
                             int &next_g, float &gain_g, int &next_c, float &gain_c)
{
    const float vcur = __fmul_rn(w, val);
    next_g = -1; gain_g = 0.0f; next_c = -1; gain_c = 0.0f;
    for (int g2 = gi + 1; g2 < sp.nG; ++g2) {
        const float v = hc[hc_idx(sp, j, g2, ci)].val;
        if (v > val) {
            next_g = g2;
            gain_g = __fdiv_rn(__fsub_rn(__fmul_rn(w, v), vcur), float(sp.g_levels[g2] - sp.g_levels[gi]));
            break;
        }
    }
    if (ci + 1 < sp.nC) {
        const float v = hc[hc_idx(sp, j, gi, ci + 1)].val;
        const float gn = __fdiv_rn(__fsub_rn(__fmul_rn(w, v), vcur), float(sp.c_levels[ci + 1] - sp.c_levels[ci]));
        if (gn > 0.0f) { next_c = ci + 1; gain_c = gn; }
    }
}

// placement requirements of a slot's candidates (see SlotC)
__device__ SlotC make_slotc(const Space &sp, const int32_t *gl, const int32_t *clv, int gi, int ci, int next_g, int next_c)
{
    SlotC s;
    const int g = gl[gi], c = clv[ci];
    s.gkind = K_NONE; s.ckind = K_NONE; s.gidx = 0; s.cidx = uint8_t(gi < sp.n_small ? gi : 0);
    s.dg = 0; s.need = 0; s.dc = 0; s.c = int16_t(c); s.c2 = 0; s.g = int16_t(g);
    if (next_g >= 0) {
        const int g2 = gl[next_g];
        if (g2 <= sp.Gn) { s.gkind = K_SINGLE; s.dg = int16_t(g2 - g); s.gidx = uint8_t(next_g); }
        else {
            const int k2 = g2 >> sp.log2Gn;
            if (cdiv_k(c, k2) <= sp.Cn) {
                if (g >= sp.Gn) { s.gkind = K_MULTI_WHOLE; s.need = int16_t(k2 - (g >> sp.log2Gn)); }
                else { s.gkind = K_MULTI_PART; s.need = int16_t(k2); }
            }
        }
    }
    if (next_c >= 0) {
        const int c2 = clv[next_c];
        s.c2 = int16_t(c2);
        if (g <= sp.Gn) { s.ckind = K_SINGLE; s.dc = int16_t(c2 - c); }
        else { const int k = g >> sp.log2Gn; if (cdiv_k(c2, k) <= sp.Cn) s.ckind = K_MULTI_WHOLE; }
    }
    return s;
}

// What a job wants next once it holds (gi, ci) with the curve's value there: its weighted gains, the GPU level
// the GPU gain refers to and what both candidates need in order to be placeable.  None of it depends on the
// cluster, so it is worked out for every (job, gi, ci) before the round and an increment that is committed in a
// batch reads one 32-byte record instead of a column of the curve.
struct __align__(16) Trans { float gain_g, gain_c; int32_t next_g, next_c; SlotC need; };
static_assert(sizeof(Trans) == 32, "two 16-byte loads");

// ---- prepare: one CTA per job.  First the curve entries at the top memory level with the plan's first feasible
// level (16 bytes each; their values also go to shared memory), then the transition records from those values.
__global__ void __launch_bounds__(256)
round_prepare_kernel(const __grid_constant__ Space sp, const rubick_job *__restrict__ jobs, const float *__restrict__ cv,
                     const int32_t *__restrict__ cp, const int32_t *__restrict__ cg, const uint32_t *__restrict__ feas,
                     HotCurve *__restrict__ hc, Trans *__restrict__ tr, const int4 *__restrict__ top)
{
    __shared__ float sval[RUBICK_MAX_G_LEVELS * RUBICK_MAX_C_LEVELS];
    const int j = blockIdx.x;
    const int per_job = sp.nG * sp.nC;
    const size_t first = size_t(j) * per_job;
    for (int e = threadIdx.x; e < per_job; e += blockDim.x) {
        const int gi = e / sp.nC;
        const size_t o = (first + e) * sp.nM + (sp.nM - 1);
        HotCurve h;
        if (top) {
            // the producer of the tables left their top memory level packed: 16 bytes instead of three 128-byte lines
            const int4 t = __ldg(top + first + e);
            h.val = __int_as_float(t.x); h.plan = t.y; h.ok = t.z == sp.g_levels[gi];
        } else {
            h.val = __ldg(cv + o); h.plan = __ldg(cp + o);
            h.ok = __ldg(cg + o) == sp.g_levels[gi];
        }
        h.f = -1;
        if (h.plan >= 0 && h.plan < sp.P) h.f = __ffs(__ldg(feas + size_t(j) * sp.P + h.plan)) - 1;
        int4 v; v.x = __float_as_int(h.val); v.y = h.plan; v.z = h.f; v.w = h.ok;
        reinterpret_cast<int4 *>(hc)[first + e] = v;
        sval[e] = h.val;
    }
    __syncthreads();
    const float w = jobs[j].w;
    for (int e = threadIdx.x; e < per_job; e += blockDim.x) {
        const int gi = e / sp.nC, ci = e - gi * sp.nC;
        Trans t; t.gain_g = 0.0f; t.gain_c = 0.0f; t.next_g = -1; t.next_c = -1;
        const float val = sval[e];
        if (val > 0.0f) {
            const float vcur = __fmul_rn(w, val);
            for (int g2 = gi + 1; g2 < sp.nG; ++g2) {
                const float x = sval[g2 * sp.nC + ci];
                if (x > val) {
                    t.next_g = g2;
                    t.gain_g = __fdiv_rn(__fsub_rn(__fmul_rn(w, x), vcur), float(sp.g_levels[g2] - sp.g_levels[gi]));
                    break;
                }
            }
            if (ci + 1 < sp.nC) {
                const float gn = __fdiv_rn(__fsub_rn(__fmul_rn(w, sval[e + 1]), vcur), float(sp.c_levels[ci + 1] - sp.c_levels[ci]));
                if (gn > 0.0f) { t.next_c = ci + 1; t.gain_c = gn; }
            }
        }
        t.need = make_slotc(sp, sp.g_levels, sp.c_levels, gi, ci, t.next_g, t.next_c);
        int4 lo, hi;
        lo.x = __float_as_int(t.gain_g); lo.y = __float_as_int(t.gain_c); lo.z = t.next_g; lo.w = t.next_c;
        hi = *reinterpret_cast<const int4 *>(&t.need);
        reinterpret_cast<int4 *>(tr + first + e)[0] = lo;
        reinterpret_cast<int4 *>(tr + first + e)[1] = hi;
    }
}

// The two increments of a running job under the present cluster state: the keys of those that have a place
// (0 = none) and the larger key among those that have a gain but no place.  w_node = the word of the job's node.
__device__ __forceinline__ void slot_keys(const Space &sp, const Views &v, int n_empty, const SlotA &a, const SlotC &q, int w_node,
                                          uint32_t &kg, uint32_t &kc, uint32_t &blocked)
{
    const int fg = fg_of(w_node), fc = fc_of(w_node);
    const int mg = v.maxc[q.gidx], mc = v.maxc[q.cidx];
    const bool part_empty = fg + q.g == sp.Gn;
    const bool ok_g = a.gain_g > 0.0f
                      && (q.gkind == K_SINGLE ? (fg >= q.dg || mg >= q.c)
                          : q.gkind == K_MULTI_WHOLE ? n_empty >= q.need
                          : q.gkind == K_MULTI_PART ? n_empty + int(part_empty) >= q.need : false);
    const bool ok_c = a.gain_c > 0.0f && (q.ckind == K_SINGLE ? (fc >= q.dc || mc >= q.c2) : q.ckind == K_MULTI_WHOLE);
    kg = ok_g ? (0x80000000u | __float_as_uint(a.gain_g)) : 0u;
    kc = ok_c ? __float_as_uint(a.gain_c) : 0u;
    blocked = 0u;
    if (!ok_g && a.gain_g > 0.0f) blocked = 0x80000000u | __float_as_uint(a.gain_g);
    if (!ok_c && a.gain_c > 0.0f) blocked = max(blocked, __float_as_uint(a.gain_c));
}

// The same for values every lane holds alike (a chain of commits): the branches are uniform, so only the tests the
// job's kinds of increment need are executed.
__device__ __forceinline__ void slot_keys_uniform(const Space &sp, const Views &v, int n_empty, const SlotA &a, const SlotC &q, int w_node,
                                                  uint32_t &placed, uint32_t &blocked)
{
    placed = 0u; blocked = 0u;
    const int fg = fg_of(w_node), fc = fc_of(w_node);
    if (a.gain_g > 0.0f) {
        bool ok = false;
        if (q.gkind == K_SINGLE) ok = fg >= q.dg || v.maxc[q.gidx] >= q.c;
        else if (q.gkind == K_MULTI_PART) ok = n_empty + int(fg + q.g == sp.Gn) >= q.need;
        else if (q.gkind == K_MULTI_WHOLE) ok = n_empty >= q.need;
        const uint32_t k = 0x80000000u | __float_as_uint(a.gain_g);
        if (ok) placed = k; else blocked = k;
    }
    if (a.gain_c > 0.0f) {
        bool ok = false;
        if (q.ckind == K_SINGLE) ok = fc >= q.dc || v.maxc[q.cidx] >= q.c2;
        else ok = q.ckind == K_MULTI_WHOLE;
        const uint32_t k = __float_as_uint(a.gain_c);
        if (ok) placed = max(placed, k); else blocked = max(blocked, k);
    }
}

// What a batch of increments needs to know about one offered candidate: can its commit be worked out without looking
// for a node (it stays where it is), does it succeed, what it changes on its node, and the largest key the job could
// offer afterwards.  The slot the job would have afterwards goes to `stage` (three 16-byte words).
struct BatchOut {
    bool elig, ok, maxc, multi;       // worked out here | the commit succeeds | maxc[] may change | the job holds whole nodes
    int slot, node, type, dgc, k;     // slot, (first) node, GPU increment?, what the node loses (GPUs << 16 | cores, or cores per node), nodes held
    int64_t dm;                       // memory the node (each node) loses
    uint32_t bound;
};

__device__ __forceinline__ void batch_candidate(const Space &sp, const Views &v, const HotCurve *__restrict__ hc, const void *tr_,
                                                int n_empty, bool saturated, const int (&mx_r)[4], const int (&gl_r)[4],
                                                uint32_t key, uint32_t pay, int j, int4 *stage, BatchOut &o)
{
    const Trans *tr = static_cast<const Trans *>(tr_);
    o.elig = o.ok = o.maxc = o.multi = false;
    o.slot = 0; o.node = -1; o.type = 0; o.dgc = 0; o.k = 1; o.dm = 0; o.bound = 0u;
    if (key == 0u || (pay & 0x80000000u)) return;
    const int s = int(pay);
    const SlotA a = v.sa[s];
    const int type_gpu = int(key >> 31);
    const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
    const int gi2 = type_gpu ? pk_next_gi(a.packed) : gi, ci2 = type_gpu ? ci : ci + 1;
    const int g = v.gl[gi], c = v.clv[ci], g2 = v.gl[gi2], c2 = v.clv[ci2];
    const int w_old = v.gc[a.node];
    // stays where it is: room on its own node, or more cores on the whole nodes it already holds
    const bool multi = g > sp.Gn;
    const int k = multi ? g >> sp.log2Gn : 1;
    const bool stays = multi ? (!type_gpu && cdiv_k(c2, k) <= sp.Cn)
                             : (g2 <= sp.Gn && fg_of(w_old) >= g2 - g && fc_of(w_old) >= c2 - c);
    if (!stays) return;
    // everything the commit and the new gains can need, in one wave of loads
    const size_t off = hc_idx(sp, j, gi2, ci2);
    const int4 b4 = *reinterpret_cast<const int4 *>(v.sb + s);
    const int4 c4 = *reinterpret_cast<const int4 *>(hc + off);
    const int4 t_lo = reinterpret_cast<const int4 *>(tr + off)[0];
    const int4 t_hi = reinterpret_cast<const int4 *>(tr + off)[1];
    SlotB b; b.val = __int_as_float(b4.x); b.plan = b4.y; b.f_level = b4.z; b.w = __int_as_float(b4.w);
    HotCurve cand; cand.val = __int_as_float(c4.x); cand.plan = c4.y; cand.f = c4.z; cand.ok = c4.w;
    SlotA na; SlotB nb; SlotC nq;
    na.gain_g = na.gain_c = 0.0f; na.packed = 0u; na.node = -1;
    nb.val = 0.0f; nb.plan = -1; nb.f_level = 0; nb.w = 0.0f;
    nq.gkind = nq.ckind = K_NONE; nq.gidx = nq.cidx = 0; nq.dg = nq.need = nq.dc = nq.c = nq.c2 = nq.g = 0;
    const int64_t m_cur = v.ml[b.f_level];
    const int64_t avail = multi ? sp.Mn * k : v.free_m[a.node] + m_cur;     // whole nodes: k shares of a node
    // levels ascend: the highest level that fits is below 0 / at least cand.f exactly when
    // level 0 / level cand.f itself does not fit / fits
    const bool none_fits = v.ml[0] > avail;
    const bool cand_fits = cand.plan >= 0 && cand.f >= 0 && cand.f < sp.nM && v.ml[cand.f >= 0 && cand.f < sp.nM ? cand.f : 0] <= avail;
    o.multi = multi; o.k = k;
    bool fz_g = pk_fz_g(a.packed), fz_c = pk_fz_c(a.packed);
    o.slot = s; o.node = a.node; o.type = type_gpu;
    if (none_fits) { o.elig = true; o.ok = false; }
    else if (cand_fits) {
        o.elig = true;
        o.ok = cand.plan < sp.P && cand.val > 0.0f && cand.ok != 0 && cand.val > b.val;
    }
    if (o.elig && o.ok) {
        // the new gains and placement needs are those of the record of (gi2, ci2): the value committed is the curve's
        na.gain_g = fz_g ? 0.0f : __int_as_float(t_lo.x); na.gain_c = fz_c ? 0.0f : __int_as_float(t_lo.y);
        na.packed = pack(gi2, ci2, t_lo.z, fz_g, fz_c); na.node = a.node;
        nb.val = cand.val; nb.plan = cand.plan; nb.f_level = cand.f; nb.w = b.w;
        nq = *reinterpret_cast<const SlotC *>(&t_hi);
        if (multi) {
            // per-node shares of cores and memory on each of the k nodes (they hold no free GPU, so maxc[] cannot change)
            o.dgc = cdiv_k(c2, k) - cdiv_k(c, k);
            o.dm = cdiv64_k(v.ml[cand.f], k) - cdiv64_k(m_cur, k);
        } else {
            o.dgc = ((g2 - g) << 16) + (c2 - c);
            o.dm = v.ml[cand.f] - m_cur;
        }
        // can maxc[] change?  (the node only loses GPUs / cores)
        const int w_new = w_old - o.dgc;
        if (!multi && !saturated) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int ot = fg_of(w_old) >= gl_r[x] ? fc_of(w_old) : -1, nt = fg_of(w_new) >= gl_r[x] ? fc_of(w_new) : -1;
                o.maxc = o.maxc || (ot == mx_r[x] && nt < ot);
            }
            for (int i = 4; i < sp.n_small; ++i) {
                const int glv = v.gl[i], mx = v.maxc[i];
                const int ot = fg_of(w_old) >= glv ? fc_of(w_old) : -1, nt = fg_of(w_new) >= glv ? fc_of(w_new) : -1;
                o.maxc = o.maxc || (ot == mx && nt < ot);
            }
        }
    } else if (o.elig) {
        // rejected: the (job, type) pair is frozen, the other increment stays as it is
        if (type_gpu) { fz_g = true; } else { fz_c = true; }
        na = a; nb = b; nq = v.sc[s];
        if (type_gpu) na.gain_g = 0.0f; else na.gain_c = 0.0f;
        na.packed = pack(gi, ci, pk_next_gi(a.packed), fz_g, fz_c);
    }
    if (o.elig) {
        // the job's own next candidates, if they could be placed (maxc[] can only have
        // shrunk by then, so testing against the present table errs on the safe side)
        const int w_new = w_old - o.dgc;
        const int fg = fg_of(w_new), fc = fc_of(w_new);
        const bool pg = na.gain_g > 0.0f
                        && (nq.gkind == K_SINGLE ? (fg >= nq.dg || v.maxc[nq.gidx] >= nq.c)
                            : nq.gkind == K_MULTI_WHOLE ? n_empty >= nq.need
                            : nq.gkind == K_MULTI_PART ? n_empty + int(fg + nq.g == sp.Gn) >= nq.need : false);
        const bool pc = na.gain_c > 0.0f && (nq.ckind == K_SINGLE ? (fc >= nq.dc || v.maxc[nq.cidx] >= nq.c2) : nq.ckind == K_MULTI_WHOLE);
        const uint32_t bg = pg ? (0x80000000u | __float_as_uint(na.gain_g)) : 0u;
        const uint32_t bc = pc ? __float_as_uint(na.gain_c) : 0u;
        o.bound = bg > bc ? bg : bc;
        stage[0] = make_int4(__float_as_int(na.gain_g), __float_as_int(na.gain_c), int(na.packed), na.node);
        stage[1] = make_int4(__float_as_int(nb.val), nb.plan, nb.f_level, __float_as_int(nb.w));
        stage[2] = *reinterpret_cast<const int4 *>(&nq);
    }
}

// warps 0 and 1 meet at barriers of their own (the block's barrier is number 0)
__device__ __forceinline__ void pair_barrier(int id) { asm volatile("bar.sync %0, 64;" :: "r"(id) : "memory"); }

// One warp's share of a batch: every lane whose candidate was taken stores what its commit changes (its node, its slot,
// the flags that make the scanning warps look again) and requests the records of the job's next candidates; jobs on whole
// nodes have every node they own updated by the whole warp.  -> may maxc[] have changed?
__device__ __forceinline__ bool batch_apply(const Space &sp, const Views &v, Shared &sh, const HotCurve *hc, const void *tr, int32_t *step_log,
                                            int N, const int4 *stage, bool taken, const BatchOut &o, int j, int log_pos, int lane)
{
    const unsigned FULL = 0xffffffffu;
    if (taken) {
        if (o.ok && !o.multi) { v.gc[o.node] -= o.dgc; v.free_m[o.node] -= o.dm; }
        const int4 na4 = stage[0];
        *reinterpret_cast<int4 *>(v.sa + o.slot) = na4;
        *reinterpret_cast<int4 *>(v.sb + o.slot) = stage[1];
        *reinterpret_cast<int4 *>(v.sc + o.slot) = stage[2];
        sh.dirty[dirty_of(o.slot)] = 1;
        if (o.ok && !o.multi) atomicOr(&v.tb[o.node >> 5], 1u << (o.node & 31));
        if (step_log) step_log[log_pos] = (j << 2) | ((o.type ? 0 : 1) << 1) | int(o.ok);
        if (o.ok) {
            const uint32_t pk = uint32_t(na4.z);
            const int ng_ = pk_next_gi(pk), gi_ = pk_gi(pk), ci_ = pk_ci(pk);
            if (__int_as_float(na4.x) > 0.0f && ng_ >= 0) prefetch_target(sp, hc, tr, j, ng_, ci_);
            if (__int_as_float(na4.y) > 0.0f && ci_ + 1 < sp.nC) prefetch_target(sp, hc, tr, j, gi_, ci_ + 1);
        }
    }
    // jobs on whole nodes: every node they own changes its share (no other job lives there)
    unsigned mm = __ballot_sync(FULL, taken && o.ok && o.multi);
    while (mm) {
        const int src = __ffs(mm) - 1;
        mm &= mm - 1;
        const int oj = __shfl_sync(FULL, j, src), dc = __shfl_sync(FULL, o.dgc, src);
        const long long dm = __shfl_sync(FULL, (long long)o.dm, src);
        const int on = __shfl_sync(FULL, o.node, src), ok_ = __shfl_sync(FULL, o.k, src);
        const int nn = on + lane;
        const bool own = lane < ok_ && nn < N && v.owner[nn] == oj;
        if (__popc(__ballot_sync(FULL, own)) == ok_) {           // its nodes are on .. on + k - 1
            if (own) { v.gc[nn] -= dc; v.free_m[nn] -= dm; }
        } else {
            for (int n = lane; n < N; n += 32)
                if (v.owner[n] == oj) { v.gc[n] -= dc; v.free_m[n] -= dm; }
        }
    }
    return __any_sync(FULL, taken && o.ok && o.maxc);
}

// One candidate staged for a chain of commits: everything its commit and its new gains can need.
//   b       value, plan, memory level and weight the job has (class entries: only the weight)
//   cand    curve entry of the target at the top memory level;  t_lo: first half of the target's transition record
//   m       x = selection key | y = job | z = slot (-1: an unallocated job) | w = target gi | ci << 8 | GPU increment << 16
//           | the usual commit applies << 17
//   cur     x = what the job holds, y = what it wants (GPUs << 16 | cores), z = its node (-1: none)
//   mem     x = memory it holds, y = memory of the target's entry (0 when that entry names no level)
//   na, nb, nq   its slot once the target's entry is committed as it stands
struct __align__(16) ChainRec { int4 m, cur; longlong2 mem; int4 na, nb, nq, b, cand, t_lo; };
constexpr int CHAIN_SLOTS = N_GROUPS - 1;    // the candidates the scanning warps offer
constexpr int CLAIMS = 512;                  // entries of the table that finds candidates of a batch on the same node
constexpr int CHAIN_CLS = 16;                // entries of the best class of unallocated jobs staged per turn
static_assert(CHAIN_CLS < 32, "lane CHAIN_CLS fetches the key behind the staged entries");

struct RoundArgs {
    const rubick_job *jobs; int J;
    const float *cv; const int32_t *cp; const int32_t *cg; const uint32_t *feas;
    int N, max_steps;
    rubick_assignment *out; rubick_node *node_out; int32_t *step_log;
    const int32_t *is_guar; const HotCurve *hc; const Trans *tr; const u64 *keys; const float *sorted_w; int n_pad; const PhaseA *pa;
    int32_t *glist;
    SlotA *sa_g; SlotB *sb_g; SlotC *sc_g; int32_t *sj_g; int slots_in_smem; int slot_cap;
    const int32_t *quota; int n_tenants;      // per tenant: GPUs, cores (n_tenants = 0: no quotas)
    uint32_t *status; int32_t *steps_out;
};

constexpr int SLOT_BYTES = int(sizeof(SlotA) + sizeof(SlotC)) + 4;     // per running job in shared memory

// warp-wide selection: largest key, lowest job among equal keys (key 0 = nothing)
__device__ __forceinline__ int warp_select(uint32_t &key, int &j, uint32_t &pay, unsigned mask = 0xffffffffu)
{
    const uint32_t m = __reduce_max_sync(mask, key);
    const int jm = __reduce_min_sync(mask, (key == m && m) ? j : 0x7fffffff);
    const unsigned b = __ballot_sync(mask, key == m && j == jm);
    const int src = b ? __ffs(b) - 1 : __ffs(mask) - 1;
    pay = __shfl_sync(mask, pay, src);
    key = m; j = jm;
    return src;                                   // the lane that held the winner
}

__global__ void __launch_bounds__(RT, 1)
greedy_round_fast_kernel(const __grid_constant__ Space sp, const __grid_constant__ RoundArgs A)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ Shared sh;
    // Phase A: pa_fail[gi * nC + ci] = number of jobs placed when a job with these target levels last found no node
    // or a node without memory for any level; while nothing else has been placed since, the next one fares the same
    // (shares its memory with what only Phase B uses)
    constexpr size_t PA_BYTES = (size_t(RUBICK_MAX_G_LEVELS) * RUBICK_MAX_C_LEVELS + 2 * RUBICK_MAX_TENANTS) * 4;
    constexpr size_t PB_BYTES = sizeof(ChainRec) * (CHAIN_SLOTS + CHAIN_CLS) + size_t(N_CAND) * 48 + size_t(CLAIMS) * 8 + 32 * 32;
    __shared__ __align__(16) unsigned char phase_buf[PA_BYTES > PB_BYTES ? PA_BYTES : PB_BYTES];
    int *pa_fail = reinterpret_cast<int *>(phase_buf);
    // Phase B: bit t set = the last head of class t was placed; the next one is then tried directly instead of
    // being looked at first as the start of a run of failing heads (either way gives the same steps)
    __shared__ uint32_t cls_went[RUBICK_MAX_G_LEVELS * RUBICK_MAX_C_LEVELS / 32];
    int32_t *rem_q = pa_fail + RUBICK_MAX_G_LEVELS * RUBICK_MAX_C_LEVELS;      // what is left of every tenant's quota: GPUs, cores
    // Phase B: the candidates of a chain of commits, in the rule's order; the slots the candidates of a batch will have;
    // the table that finds candidates of a batch on the same node (highest key, lowest job among equal keys)
    ChainRec *chain = reinterpret_cast<ChainRec *>(phase_buf);
    int4 *bst = reinterpret_cast<int4 *>(phase_buf + sizeof(ChainRec) * (CHAIN_SLOTS + CHAIN_CLS));
    uint32_t *claim_k = reinterpret_cast<uint32_t *>(phase_buf + sizeof(ChainRec) * (CHAIN_SLOTS + CHAIN_CLS) + size_t(N_CAND) * 48);
    int32_t *claim_j = reinterpret_cast<int32_t *>(claim_k + CLAIMS);
    int4 *bres = reinterpret_cast<int4 *>(claim_j + CLAIMS);      // what warp 1 found out about the second candidate of every lane
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = A.N, J = A.J;
    const int n_cls = sp.nG * sp.nC;

    Views v;
    v.N = N; v.N_pad = (N + 127) & ~127;
    unsigned char *p = smem_raw;
    v.gc = reinterpret_cast<int32_t *>(p); p += size_t(v.N_pad) * 4;            // 16-byte aligned: read as int4
    v.free_m = reinterpret_cast<int64_t *>(p); p += size_t(N) * 8;
    v.cls_top = reinterpret_cast<u64 *>(p); p += size_t(n_cls) * 8;
    int64_t *ml_s = reinterpret_cast<int64_t *>(p); p += size_t(RUBICK_MAX_M_LEVELS) * 8;
    v.owner = reinterpret_cast<int32_t *>(p); p += size_t(N) * 4;
    v.cls_ptr = reinterpret_cast<int32_t *>(p); p += size_t(n_cls) * 4;
    v.cls_end = reinterpret_cast<int32_t *>(p); p += size_t(n_cls) * 4;
    v.cls_w = reinterpret_cast<float *>(p); p += size_t(n_cls) * 4;
    v.ccls = reinterpret_cast<int32_t *>(p); p += size_t(n_cls) * 4;
    v.maxc = reinterpret_cast<int32_t *>(p); p += size_t(RUBICK_MAX_G_LEVELS) * 4;
    int32_t *gl_s = reinterpret_cast<int32_t *>(p); p += size_t(RUBICK_MAX_G_LEVELS) * 4;
    int32_t *cl_s = reinterpret_cast<int32_t *>(p); p += size_t(RUBICK_MAX_C_LEVELS) * 4;
    uint32_t *tb_s = reinterpret_cast<uint32_t *>(p); p += size_t(v.N_pad / 32) * 4;
    v.gl = gl_s; v.clv = cl_s; v.ml = ml_s; v.tb = tb_s;
    p = smem_raw + ((size_t(p - smem_raw) + 15) & ~size_t(15));
    if (A.slots_in_smem) {
        v.sa = reinterpret_cast<SlotA *>(p); p += size_t(A.slot_cap) * sizeof(SlotA);
        v.sc = reinterpret_cast<SlotC *>(p); p += size_t(A.slot_cap) * sizeof(SlotC);
        v.sj = reinterpret_cast<int32_t *>(p);
    } else { v.sa = A.sa_g; v.sc = A.sc_g; v.sj = A.sj_g; }
    // value / plan / memory level / weight: touched only by commits, kept in global memory (shared memory taken for them
    // would come out of the L1 cache the curve entries and transition records are requested into)
    v.sb = A.sb_g;

    // ---- set-up ---------------------------------------------------------------------------------
    for (int n = tid; n < v.N_pad; n += RT) v.gc[n] = n < N ? ((sp.Gn << 16) | sp.Cn) : 0;
    for (int n = tid; n < N; n += RT) { v.free_m[n] = sp.Mn; v.owner[n] = -1; }
    for (int t = tid; t < n_cls; t += RT) { v.cls_ptr[t] = 0; v.cls_end[t] = 0; v.cls_top[t] = 0ull; v.cls_w[t] = 0.0f; }
    if (tid < sp.nG) gl_s[tid] = sp.g_levels[tid];
    if (tid < sp.nC) cl_s[tid] = sp.c_levels[tid];
    if (tid < sp.nM) ml_s[tid] = sp.m_levels[tid];
    for (int i = tid; i < v.N_pad / 32; i += RT) tb_s[i] = 0u;
    if (tid < sp.n_small) v.maxc[tid] = sp.Cn;                              // every node is empty
    if (tid < N_CAND) { sh.dirty[tid] = 1; sh.red_key[tid] = 0u; sh.red_j[tid] = 0x7fffffff; sh.red_pay[tid] = 0u; sh.red_key2[tid] = 0u; }
    if (tid < RUBICK_MAX_G_LEVELS) sh.ff_pos[tid] = 0;
    for (int t = tid; t < n_cls; t += RT) pa_fail[t] = -1;
    for (int t = tid; t < RUBICK_MAX_G_LEVELS * RUBICK_MAX_C_LEVELS / 32; t += RT) cls_went[t] = 0u;
    for (int i = tid; i < 2 * A.n_tenants; i += RT) rem_q[i] = A.quota[i];
    if (tid == 0) {
        sh.n_empty = N; sh.n_slots = 0; sh.steps = 0; sh.capped = 0; sh.stop = 0; sh.n_guar = 0; sh.n_ccls = 0;
        sh.ver = 0; sh.maxc_dirty = 1; sh.empty_lo = 0; sh.pa_commits = 0;
    }
    __syncthreads();

    // class segments of the sorted keys: a class starts where the class field changes
    for (int i = tid; i < A.n_pad; i += RT) {
        const u64 k = A.keys[i];
        const u64 kp = i ? A.keys[i - 1] : 0ull;
        if (k && (i == 0 || key_class(kp) != key_class(k))) {
            const int cls = key_class(k);
            const int t = (cls >> 6) * sp.nC + (cls & 63);
            v.cls_ptr[t] = i; v.cls_top[t] = k; v.cls_w[t] = A.sorted_w[i];
        }
        if (i && kp && (!k || key_class(kp) != key_class(k))) {
            const int cls = key_class(kp);
            v.cls_end[(cls >> 6) * sp.nC + (cls & 63)] = i;
        }
        if (i == A.n_pad - 1 && k) {
            const int cls = key_class(k);
            v.cls_end[(cls >> 6) * sp.nC + (cls & 63)] = A.n_pad;
        }
    }
    // the ordered list of guaranteed jobs: every warp owns a contiguous stretch of the job indices, counts its
    // marks 32 at a time, and writes them behind those of the warps before it
    {
        const int per_warp = (((J + RW - 1) / RW) + 31) & ~31;
        const int w0 = min(warp * per_warp, J), w1 = min(w0 + per_warp, J);
        int cnt = 0;
        for (int base = w0; base < w1; base += 32)
            cnt += __popc(__ballot_sync(0xffffffffu, base + lane < w1 && A.is_guar[base + lane] != 0));
        if (lane == 0) sh.scan_cnt[warp] = cnt;
        __syncthreads();
        if (warp == 0) {
            int wsum = lane < RW ? sh.scan_cnt[lane] : 0;
#pragma unroll
            for (int s = 1; s < 32; s <<= 1) { const int o = __shfl_up_sync(0xffffffffu, wsum, s); if (lane >= s) wsum += o; }
            if (lane < RW) sh.scan_cnt[lane] = wsum;
            if (lane == 31) sh.n_guar = wsum;
            // compact list of the classes that have members
            int n_c = 0;
            for (int base = 0; base < n_cls; base += 32) {
                const int t = base + lane;
                const bool has = t < n_cls && v.cls_top[t] != 0ull;
                const unsigned b = __ballot_sync(0xffffffffu, has);
                if (has) v.ccls[n_c + __popc(b & ((1u << lane) - 1u))] = t | ((t / sp.nC) << 16) | ((t % sp.nC) << 24);
                n_c += __popc(b);
            }
            if (lane == 0) sh.n_ccls = n_c;
        }
        __syncthreads();
        int pos = warp ? sh.scan_cnt[warp - 1] : 0;
        for (int base = w0; base < w1; base += 32) {
            const bool g = base + lane < w1 && A.is_guar[base + lane] != 0;
            const unsigned b = __ballot_sync(0xffffffffu, g);
            if (g) A.glist[pos + __popc(b & ((1u << lane) - 1u))] = base + lane;
            pos += __popc(b);
        }
    }
    __syncthreads();

    // ---- Phase A: guaranteed minima in job order (warp 0) ------------------------------------------
    if (warp == 0) {
        const int ng = sh.n_guar;
        // the phase's counters live in registers (every lane holds the same values) and go back to shared memory
        // around the calls that use them there and at the end
        int commits = sh.pa_commits, n_slots_r = sh.n_slots, n_empty_r = sh.n_empty;
        // lanes fetch 32 list entries at once; they are used one after another.  The records of the next 32 and
        // the list entries of the 32 after them are requested before this batch is worked on.
        int jl = lane < ng ? A.glist[lane] : -1;
        int jl_next = 32 + lane < ng ? A.glist[32 + lane] : -1;
        int4 a0 = make_int4(-1, 0, 0, -1), a1 = make_int4(-1, 0, 0, 0);
        if (jl >= 0) { a0 = reinterpret_cast<const int4 *>(A.pa + jl)[0]; a1 = reinterpret_cast<const int4 *>(A.pa + jl)[1]; }
        for (int base = 0; base < ng; base += 32) {
            const int idx = base + lane;
            int4 n0 = make_int4(-1, 0, 0, -1), n1 = make_int4(-1, 0, 0, 0);
            if (jl_next >= 0) { n0 = reinterpret_cast<const int4 *>(A.pa + jl_next)[0]; n1 = reinterpret_cast<const int4 *>(A.pa + jl_next)[1]; }
            const int jl_after = base + 64 + lane < ng ? A.glist[base + 64 + lane] : -1;
            // Free resources only shrink during this phase, so a job that cannot be placed now never can:
            // every lane tests its own job against the present tables and only the others take a turn.
            bool may = false;
            int need_l = 0, tag_l = 0;              // (GPUs << 16 | cores) of the job's minimum; index of its failure mark | GPU level << 12
            if (idx < ng && a0.x >= 0) {
                const int g2 = v.gl[a0.x], c2 = v.clv[a0.y];
                need_l = (g2 << 16) | c2; tag_l = (a0.x * sp.nC + a0.y) | (a0.x << 12);
                if (g2 <= sp.Gn) may = v.maxc[a0.x] >= c2;
                else { const int k2 = g2 >> sp.log2Gn; may = (c2 + k2 - 1) / k2 <= sp.Cn && n_empty_r >= k2; }
                may = may && pa_fail[tag_l & 0xfff] != commits;
            }
            unsigned todo = __ballot_sync(0xffffffffu, may);
            // what a turn needs of its job beyond the cluster's state, worked out by the job's lane: is the curve entry
            // of the target usable as it stands (a plan that runs, with the level's own GPU count), and the memory it takes
            const bool entry_ok = a0.w >= 0 && a0.w < sp.P && __int_as_float(a0.z) > 0.0f && a1.y != 0 && a1.x >= 0 && a1.x < sp.nM;
            const long long m_need_l = entry_ok ? v.ml[a1.x] : 0;
            if (entry_ok) tag_l |= 1 << 20;
            // Turns run on all lanes alike (shuffles hand out what the turn needs of the job's record, every lane reads and
            // writes the same shared-memory words, so each lane sees its own stores and the warp never has to synchronise).
            // The usual turn -- a job that fits one node, whose curve entry is usable and whose memory fits the node found
            // -- touches five words: the failure mark of its levels, the first-fit mark, the node's GPUs / cores and
            // memory; the job's lane notes the slot and the node, and writes the slot when the 32 jobs are through.
            // Anything else (whole-node minima, an entry that needs the table) goes through commit_warp.
            int my_slot = -1, my_node = -1;
            while (todo) {
                const int i = __ffs(todo) - 1;
                todo &= todo - 1;
                const int tag = __shfl_sync(0xffffffffu, tag_l, i), need = __shfl_sync(0xffffffffu, need_l, i);
                const long long m_need = __shfl_sync(0xffffffffu, m_need_l, i);
                const int cls = tag & 0xfff, gi = (tag >> 12) & 0xff;
                const bool usable = (tag >> 20) & 1;
                const int g2 = need >> 16, c2 = need & 0xffff;
                int tn = 0;
                if (A.n_tenants > 0) {     // privileged only while the minimum fits the tenant's remaining quota
                    tn = __shfl_sync(0xffffffffu, a1.w, i);
                    if (tn < 0 || tn >= A.n_tenants) continue;
                    if (rem_q[2 * tn] < g2 || rem_q[2 * tn + 1] < c2) continue;
                }
                if (pa_fail[cls] == commits) continue;              // same levels, same cluster: same outcome
                bool settled = false;
                if (g2 <= sp.Gn && usable) {
                    // no node below the mark has g2 free GPUs: if the node at the mark fits, it is the first fit
                    int mark = sh.ff_pos[gi];
                    int target = mark;
                    int w_old = target < N ? v.gc[target] : 0;
                    int64_t fm = target < N ? v.free_m[target] : 0;          // (asked for together with the node's word)
                    if (!(fg_of(w_old) >= g2 && fc_of(w_old) >= c2)) {
                        target = first_fit_from_mark(v, sh, gi, g2, c2, lane);
                        if (target < 0) { pa_fail[cls] = commits; continue; }      // no node for these levels
                        w_old = v.gc[target]; fm = v.free_m[target]; mark = sh.ff_pos[gi];
                    }
                    if (m_need <= fm) {
                        // the highest memory level that fits the node is at or above the plan's own: the entry stands
                        v.gc[target] = w_old - need;
                        v.free_m[target] = fm - m_need;
                        if (fg_of(w_old) == sp.Gn) --n_empty_r;
                        // the node at the mark has just lost the GPUs the next job of these levels would need: the mark
                        // moves on at once, and that job looks at the following node without a search
                        if (mark == target && fg_of(w_old) - g2 < g2) sh.ff_pos[gi] = target + 1;
                        if (lane == i) { my_slot = n_slots_r; my_node = target; }
                        settled = true;
                    } else if (v.ml[0] > fm) { pa_fail[cls] = commits; continue; }   // the node found has memory for no level
                }
                if (!settled) {
                    const int ci = __shfl_sync(0xffffffffu, a0.y, i), j = __shfl_sync(0xffffffffu, jl, i);
                    const float w = __int_as_float(__shfl_sync(0xffffffffu, a1.z, i));
                    HotCurve cand;
                    cand.val = __int_as_float(__shfl_sync(0xffffffffu, a0.z, i));
                    cand.plan = __shfl_sync(0xffffffffu, a0.w, i); cand.f = __shfl_sync(0xffffffffu, a1.x, i);
                    cand.ok = __shfl_sync(0xffffffffu, a1.y, i);
                    Committed cm; cm.first = -1; cm.val = cand.val; cm.plan = cand.plan; cm.f = cand.f;
                    sh.n_empty = n_empty_r;
                    __syncwarp();
                    settled = commit_warp<false, COMMIT_PHASE_A>(sp, v, sh, A.cv, A.cp, A.cg, A.feas, j, -1, 0, -1, 0.0f, 0, gi, ci, cand, false, lane, cm);
                    __syncwarp();
                    n_empty_r = sh.n_empty;
                    if (!settled) {
                        if (cm.first == -2) pa_fail[cls] = commits;
                        continue;
                    }
                    if (lane == 0) {
                        const int s = n_slots_r;
                        SlotA sa; sa.gain_g = 0.0f; sa.gain_c = 0.0f; sa.packed = pack(gi, ci, -1, false, false); sa.node = cm.first;
                        SlotB sb; sb.val = cm.val; sb.plan = cm.plan; sb.f_level = cm.f; sb.w = w;
                        v.sa[s] = sa; v.sb[s] = sb; v.sj[s] = j;
                    }
                }
                ++n_slots_r;
                ++commits;
                if (A.n_tenants > 0) {
                    const int qg = rem_q[2 * tn], qc = rem_q[2 * tn + 1];
                    rem_q[2 * tn] = qg - g2; rem_q[2 * tn + 1] = qc - c2;
                }
            }
            if (my_slot >= 0) {          // placed by the usual turn, with the curve entry as it stands
                SlotA sa; sa.gain_g = 0.0f; sa.gain_c = 0.0f; sa.packed = pack(a0.x, a0.y, -1, false, false); sa.node = my_node;
                SlotB sb; sb.val = __int_as_float(a0.z); sb.plan = a0.w; sb.f_level = a1.x; sb.w = __int_as_float(a1.z);
                v.sa[my_slot] = sa; v.sb[my_slot] = sb; v.sj[my_slot] = jl;
            }
            jl = jl_next; a0 = n0; a1 = n1; jl_next = jl_after;
        }
        // During this phase maxc[] only served as a hint that errs on the generous side (the usual turn does not
        // maintain it; free resources only shrink, so an old entry is never too small): make it exact again.
        sh.pa_commits = commits; sh.n_slots = n_slots_r; sh.n_empty = n_empty_r;
        __syncwarp();
        rebuild_maxc_warp(sp, v, lane);
    }
    __syncthreads();
    for (int i = tid; i < CLAIMS; i += RT) { claim_k[i] = 0u; claim_j[i] = 0x7fffffff; }
    // gains of the jobs placed in Phase A
    for (int s = tid; s < sh.n_slots; s += RT) {
        SlotA a = v.sa[s]; const SlotB b = v.sb[s];
        int ng_, nc_; float gg, gc;
        gains_thread(sp, A.hc, v.sj[s], b.w, pk_gi(a.packed), pk_ci(a.packed), b.val, ng_, gg, nc_, gc);
        a.gain_g = gg; a.gain_c = gc; a.packed = pack(pk_gi(a.packed), pk_ci(a.packed), ng_, false, false);
        v.sa[s] = a;
        v.sc[s] = make_slotc(sp, v.gl, v.clv, pk_gi(a.packed), pk_ci(a.packed), ng_, nc_);
    }
    __syncthreads();

    // ---- Phase B ---------------------------------------------------------------------------------------
    // Every warp leaves the best OFFER candidates among its own slots in shared memory (the last warp: the best class
    // head) and looks again only when something it depends on changed: one of its slots, a node one of its slots
    // sits on, maxc[] or the number of empty nodes.
    int my_ver = -1;
    for (;;) {
        if (sh.maxc_dirty) {                                   // uniform: written before the last barrier
            if (warp < sp.n_small) {
                const int m = max_cores_warp(v, sp.g_levels[warp], lane);
                if (lane == 0 && m != v.maxc[warp]) { v.maxc[warp] = m; atomicAdd(&sh.ver, 1); }
            }
            __syncthreads();
        }
        const int n_empty = sh.n_empty, n_slots = sh.n_slots, ver = sh.ver;
        const unsigned hm = 0xffffffffu;
        const int grp = warp < SCAN_WARPS ? OFFER * warp : CLS_G;     // index of the warp's first candidate
        bool rescan = ver != my_ver || sh.dirty[grp] != 0;
        if (warp < SCAN_WARPS) {
            if (!rescan) {
                bool hit = false;
                for (int s = tid; s < n_slots; s += SCAN_T) { const int nd = v.sa[s].node; hit = hit || ((v.tb[nd >> 5] >> (nd & 31)) & 1u); }
                rescan = __any_sync(hm, hit);
            }
            if (rescan) {
                // the two best candidates of my slots in full, of everything else only the largest key
                uint32_t k1 = 0u, k2 = 0u, rest = 0u, p1 = 0u, p2 = 0u, blk = 0u; int j1 = 0x7fffffff, j2 = 0x7fffffff;
                for (int s = tid; s < n_slots; s += SCAN_T) {
                    const SlotA a = v.sa[s];
                    const SlotC q = v.sc[s];
                    const int j = v.sj[s];
                    const int w = v.gc[a.node];
                    const int fg = fg_of(w), fc = fc_of(w);
                    const int mg = v.maxc[q.gidx], mc = v.maxc[q.cidx];
                    const bool part_empty = fg + q.g == sp.Gn;
                    const bool ok_g = a.gain_g > 0.0f
                                      && (q.gkind == K_SINGLE ? (fg >= q.dg || mg >= q.c)
                                          : q.gkind == K_MULTI_WHOLE ? n_empty >= q.need
                                          : q.gkind == K_MULTI_PART ? n_empty + int(part_empty) >= q.need : false);
                    const bool ok_c = a.gain_c > 0.0f && (q.ckind == K_SINGLE ? (fc >= q.dc || mc >= q.c2) : q.ckind == K_MULTI_WHOLE);
                    // a GPU increment outranks any CPU increment; the job's other increment is only a runner-up
                    const uint32_t kg = ok_g ? (0x80000000u | __float_as_uint(a.gain_g)) : 0u;
                    const uint32_t kc = ok_c ? __float_as_uint(a.gain_c) : 0u;
                    const uint32_t k32 = ok_g ? kg : kc;
                    if (!ok_g && a.gain_g > 0.0f) blk = max(blk, 0x80000000u | __float_as_uint(a.gain_g));
                    if (!ok_c && a.gain_c > 0.0f) blk = max(blk, __float_as_uint(a.gain_c));
                    if (k32 > k1 || (k32 == k1 && k32 && j < j1)) {
                        rest = max(rest, k2); k2 = k1; j2 = j1; p2 = p1; k1 = k32; j1 = j; p1 = uint32_t(s);
                    } else if (k32 > k2 || (k32 == k2 && k32 && j < j2)) {
                        rest = max(rest, k2); k2 = k32; j2 = j; p2 = uint32_t(s);
                    } else rest = max(rest, k32);
                    if (ok_g) rest = max(rest, kc);
                }
                // the warp's best OFFER candidates one after another (the lane that gave one puts up its own second;
                // a third of the same lane counts with what remains); then the largest key among what remains
                uint32_t o_k = 0u, o_p = 0u; int o_j = 0x7fffffff;          // lane r keeps the warp's r-th candidate
#pragma unroll
                for (int r = 0; r < OFFER; ++r) {
                    uint32_t w_k = k1, w_p = p1; int w_j = j1;
                    const int src = warp_select(w_k, w_j, w_p, hm);
                    if (lane == r) { o_k = w_k; o_j = w_j; o_p = w_p; }
                    if (lane == src && w_k != 0u) { k1 = k2; j1 = j2; p1 = p2; k2 = 0u; j2 = 0x7fffffff; }
                }
                const uint32_t key2 = __reduce_max_sync(hm, max(rest, max(k1, k2)));
                const uint32_t blkw = __reduce_max_sync(hm, blk);
                if (lane < OFFER) {
                    sh.red_key[grp + lane] = o_k; sh.red_j[grp + lane] = o_j; sh.red_pay[grp + lane] = o_p;
                    sh.red_key2[grp + lane] = lane == 0 ? key2 : (lane == 1 ? blkw : 0u);
                }
                my_ver = ver;
                if (lane == 0) sh.dirty[grp] = 0;
            }
        } else if (rescan) {
            uint32_t best = 0u, second = 0u, pay = 0u, blk = 0u; int best_j = 0x7fffffff;
            const int n_ccls = sh.n_ccls;
            for (int i = lane; i < n_ccls; i += 32) {
                const int packed = v.ccls[i];
                const int t = packed & 0xffff, gi2 = (packed >> 16) & 0xff, ci2 = (packed >> 24) & 0xff;
                const u64 k = v.cls_top[t];
                if (k) {
                    const int g2 = v.gl[gi2], c2 = v.clv[ci2];
                    bool ok;
                    if (g2 <= sp.Gn) ok = v.maxc[gi2] >= c2;
                    else { const int k2 = g2 >> sp.log2Gn; ok = (c2 + k2 - 1) / k2 <= sp.Cn && n_empty >= k2; }
                    const uint32_t k32 = ok ? (0x80000000u | key_gain_bits(k)) : 0u;
                    if (!ok) blk = max(blk, 0x80000000u | key_gain_bits(k));
                    const int j = key_job(k);
                    if (k32 > best || (k32 == best && k32 && j < best_j)) { second = best; best = k32; best_j = j; pay = 0x80000000u | uint32_t(t); }
                    else if (k32 > second) second = k32;
                }
            }
            const uint32_t mine = best;
            const int src = warp_select(best, best_j, pay);
            const uint32_t key2 = __reduce_max_sync(0xffffffffu, lane == src ? second : mine);
            const uint32_t blkw = __reduce_max_sync(0xffffffffu, blk);
            my_ver = ver;
            if (lane == 0) {
                sh.red_key[CLS_G] = best; sh.red_j[CLS_G] = best_j; sh.red_pay[CLS_G] = pay;
                sh.red_key2[CLS_G] = key2; sh.red_key2[CLS_G + 1] = blkw;
                sh.dirty[CLS_G] = 0;
            }
        }
        __syncthreads();
        if (warp == 0) {
            const unsigned FULL = 0xffffffffu;
            // two candidates a lane: those of index lane and lane + 32 (the class head is the second one of lane CLS_G - 32)
            uint32_t key_[2], pay_[2]; int j_[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) { key_[u] = sh.red_key[lane + 32 * u]; pay_[u] = sh.red_pay[lane + 32 * u]; j_[u] = sh.red_j[lane + 32 * u]; }
            const bool second_u = key_[1] > key_[0] || (key_[1] == key_[0] && key_[1] && j_[1] < j_[0]);
            uint32_t best = second_u ? key_[1] : key_[0], pay = second_u ? pay_[1] : pay_[0]; int best_j = second_u ? j_[1] : j_[0];
            const int top_lane = warp_select(best, best_j, pay);
            bool go = best != 0u;
            const int steps0 = sh.steps, room = A.max_steps - steps0;
            if (go && room <= 0) { if (lane == 0) sh.capped = 1; go = false; }
            if (lane == 0) sh.maxc_dirty = 0;
            for (int i = lane; i < v.N_pad / 32; i += 32) v.tb[i] = 0u;
            __syncwarp();

            // ---- a batch of independent increments ---------------------------------------------------------
            // Every lane holds two candidates offered by the scanning warps.  Increments that stay on their node, on pairwise
            // different nodes, commute with everything except what happens on that node, so the next few
            // picks of the sequential rule can be committed together as long as each of them still is the
            // largest candidate: larger than every key that was not offered (M), than the offered ones not yet
            // taken, and than the new candidates of the jobs taken before it.  Each lane works out the commits of
            // its own candidates first (one wave of global loads for all of them together instead of several per step).
            int n_acc = 0;
            // ---- a run of class heads that cannot be committed --------------------------------------------
            // A rejected increment changes nothing but the head of its class, so as long as the heads of that
            // class outrank every other candidate the sequential rule keeps trying them one after another
            // against the same target and the same memory level: lane i settles the i-th entry of the
            // class's sorted list, and everything before the first entry that would succeed is consumed.
            if (go && (pay & 0x80000000u) && !((cls_went[(pay & 0x7fffffffu) >> 5] >> (pay & 31u)) & 1u)) {
                const int t = int(pay & 0x7fffffffu);
                const int gi2 = t / sp.nC, ci2 = t - gi2 * sp.nC;
                const int g2 = sp.g_levels[gi2], c2 = sp.c_levels[ci2];
                // the largest key among everything but the heads of this class
                const uint32_t B = __reduce_max_sync(FULL, max(key_[0], lane + 32 == CLS_G ? sh.red_key2[CLS_G] : key_[1]));
                int k2 = 1; int64_t avail = -1;
                if (g2 <= sp.Gn) {
                    const int target = v.maxc[gi2] >= c2 ? first_fit_warp(v, g2, c2, lane) : -1;
                    if (target >= 0) avail = v.free_m[target];
                } else {
                    k2 = g2 >> sp.log2Gn;
                    if ((c2 + k2 - 1) / k2 <= sp.Cn && sh.n_empty >= k2) avail = sp.Mn;
                }
                if (avail >= 0) {
                    const unsigned fb = __ballot_sync(FULL, lane < sp.nM && v.ml[lane < sp.nM ? lane : 0] <= avail * k2);
                    const int mi = fb ? 31 - __clz(fb) : -1;
                    const int ptr = v.cls_ptr[t], end = v.cls_end[t];
                    int n_fail = 0;
                    if (mi < 0) {
                        // The node has no memory for any level: every head of the class that outranks the rest fails
                        // the same way.  The class is sorted, so they are counted by a search with 32 probes a step.
                        int lo = ptr, hi = end;          // entries before lo are in the run, entry hi (if any) is not
                        while (lo < hi) {
                            const int stride = (hi - lo + 31) / 32;
                            const int idx = lo + lane * stride;
                            const bool in = idx < hi && (0x80000000u | key_gain_bits(A.keys[idx])) > B;
                            const int c = __popc(__ballot_sync(FULL, in));
                            if (c == 0) break;
                            hi = min(lo + c * stride, hi);
                            lo += (c - 1) * stride + 1;
                        }
                        n_fail = min(lo - ptr, room);
                        if (A.step_log)
                            for (int i = lane; i < n_fail; i += 32) A.step_log[steps0 + i] = (key_job(A.keys[ptr + i]) << 2) | 0;
                    } else {
                    // RUN_U x 32 entries a turn: every lane looks at RUN_U of them, all loads of a kind in one wave
                    u64 k[RUN_U]; bool in_run[RUN_U], succ[RUN_U]; HotCurve cand[RUN_U];
#pragma unroll
                    for (int u = 0; u < RUN_U; ++u) {
                        const int idx = ptr + 32 * u + lane;
                        k[u] = idx < end ? A.keys[idx] : 0ull;
                    }
#pragma unroll
                    for (int u = 0; u < RUN_U; ++u) {
                        in_run[u] = k[u] != 0ull && (0x80000000u | key_gain_bits(k[u])) > B;
                        succ[u] = false;
                        if (in_run[u] && mi >= 0) cand[u] = load_hc(A.hc + hc_idx(sp, key_job(k[u]), gi2, ci2));
                    }
                    bool open_ = true;                          // leading entries that are in the run and fail
#pragma unroll
                    for (int u = 0; u < RUN_U; ++u) {
                        if (in_run[u] && mi >= 0) {
                            const int j = key_job(k[u]);
                            float val; int plan, f; bool okg;
                            if (cand[u].plan >= 0 && cand[u].f >= 0 && cand[u].f <= mi) { val = cand[u].val; plan = cand[u].plan; f = cand[u].f; okg = cand[u].ok != 0; }
                            else {
                                const size_t o = curve_idx(sp, j, gi2, ci2, mi);
                                val = __ldg(A.cv + o); plan = __ldg(A.cp + o); okg = __ldg(A.cg + o) == g2;
                                f = -1;
                                if (plan >= 0 && plan < sp.P) f = __ffs(__ldg(A.feas + size_t(j) * sp.P + plan)) - 1;
                            }
                            succ[u] = plan >= 0 && plan < sp.P && val > 0.0f && okg && f >= 0 && f <= mi;
                        }
                        const unsigned stop = __ballot_sync(FULL, !in_run[u] || succ[u]);
                        if (open_) { n_fail += stop ? __ffs(stop) - 1 : 32; open_ = stop == 0u; }
                    }
                    if (n_fail > room) n_fail = room;
                    if (A.step_log) {
#pragma unroll
                        for (int u = 0; u < RUN_U; ++u)
                            if (32 * u + lane < n_fail) A.step_log[steps0 + 32 * u + lane] = (key_job(k[u]) << 2) | 0;
                    }
                    }
                    if (n_fail > 0) {
                        if (lane == 0) {
                            const int np = ptr + n_fail;
                            u64 nk = 0ull; float nw = 0.0f;
                            if (np < end) { nk = A.keys[np]; nw = A.sorted_w[np]; }
                            v.cls_ptr[t] = np; v.cls_top[t] = nk; v.cls_w[t] = nw;
                            sh.dirty[CLS_G] = 1;
                            sh.steps = steps0 + n_fail;
                        }
                        n_acc = n_fail;
                    }
                }
            }
            // the batch can only start with the overall best candidate: look at it first (shared memory only)
            bool top_stays = false;
            if (go && n_acc == 0 && !(pay & 0x80000000u)) {
                bool st = false;
                if (lane == top_lane) {
                    const SlotA a = v.sa[int(pay)];
                    const int type_gpu = int(best >> 31);
                    const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
                    const int gi2 = type_gpu ? pk_next_gi(a.packed) : gi, ci2 = type_gpu ? ci : ci + 1;
                    const int g = v.gl[gi], c = v.clv[ci], g2 = v.gl[gi2], c2 = v.clv[ci2];
                    const int w_old = v.gc[a.node];
                    const int k = g > sp.Gn ? g >> sp.log2Gn : 1;
                    st = g > sp.Gn ? (!type_gpu && cdiv_k(c2, k) <= sp.Cn)
                                   : (g2 <= sp.Gn && fg_of(w_old) >= g2 - g && fc_of(w_old) >= c2 - c);
                }
                top_stays = __any_sync(FULL, st);
            }
            // Warp 1 works out the second candidate of every lane while this warp works out the first: it waits for the
            // word that says whether there is a batch, and hands its results over in shared memory.
            const bool batch = go && n_acc == 0 && top_stays;
            if (lane == 0) sh.batch_go = batch ? 1 : 0;
            pair_barrier(1);
            if (batch) {
                const uint32_t M = __reduce_max_sync(FULL, lane < 16 ? sh.red_key2[OFFER * lane] : 0u);
                // per candidate (two a lane): can its commit be worked out here, does it succeed, and what it changes;
                // the slot it has afterwards waits in shared memory (bst) until the candidate is taken
                bool elig[2], s_ok[2], s_maxc[2], s_multi[2];
                int s_slot[2], s_node[2], s_type[2], s_dgc[2], s_k[2];
                int64_t s_dm[2];
                uint32_t s_bound[2];
                {
                    // the same for every lane: while an empty node remains and every maxc[] entry is the node's core
                    // count no commit that stays on its node can change maxc[]; the first four levels in registers
                    const int n_empty = sh.n_empty;
                    const bool saturated = n_empty > 0 && __all_sync(FULL, lane >= sp.n_small || v.maxc[lane] == sp.Cn);
                    int mx_r[4], gl_r[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) { mx_r[u] = u < sp.n_small ? v.maxc[u] : -2; gl_r[u] = u < sp.n_small ? v.gl[u] : 0x7fffffff; }
                    BatchOut o;
                    batch_candidate(sp, v, A.hc, A.tr, n_empty, saturated, mx_r, gl_r, key_[0], pay_[0], j_[0], bst + 3 * lane, o);
                    elig[0] = o.elig; s_ok[0] = o.ok; s_maxc[0] = o.maxc; s_multi[0] = o.multi;
                    s_slot[0] = o.slot; s_node[0] = o.node; s_type[0] = o.type; s_dgc[0] = o.dgc; s_k[0] = o.k; s_dm[0] = o.dm; s_bound[0] = o.bound;
                }
                pair_barrier(2);
                {
                    const int4 r0 = bres[2 * lane], r1 = bres[2 * lane + 1];
                    elig[1] = r0.x & 1; s_ok[1] = (r0.x >> 1) & 1; s_maxc[1] = (r0.x >> 2) & 1; s_multi[1] = (r0.x >> 3) & 1; s_type[1] = (r0.x >> 4) & 1;
                    s_slot[1] = r0.y; s_node[1] = r0.z; s_dgc[1] = r0.w;
                    s_k[1] = r1.x; s_bound[1] = uint32_t(r1.y);
                    s_dm[1] = (int64_t(uint32_t(r1.w)) << 32) | int64_t(uint32_t(r1.z));
                }
                // Take the candidates in the order the sequential rule would: by descending key, lowest job first
                // among equal keys.  The rule goes on while the next candidate could be worked out here, sits on a
                // node of its own, and its key exceeds M and the bound of every candidate before it.  All of this
                // holds for the candidates above one threshold t: the largest of M, the keys of the candidates that
                // could not be worked out, the keys of those that share a node with a candidate ranked before them,
                // and, among what is left, every bound (a bound at or above its own key: that key).  They form a
                // prefix of the order, possibly a little shorter than the longest one; the rest waits a turn.
                u64 mine[2]; bool usable[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    // key, then lowest job, then index: all words differ
                    mine[u] = (u64(key_[u]) << 32) | (key_[u] ? u64(uint32_t(KEY_JOB_MASK) - uint32_t(j_[u])) << 6 : 0ull) | u64(63 - lane - 32 * u);
                    sh.sel[lane + 32 * u] = mine[u];
                    usable[u] = key_[u] != 0u && elig[u];
                }
                uint32_t t = __reduce_max_sync(FULL, max(key_[0] != 0u && !elig[0] ? key_[0] : 0u, key_[1] != 0u && !elig[1] ? key_[1] : 0u));
                if (M > t) t = M;
                // Which candidates sit on a node together with one ranked before them?  Every candidate puts its key up
                // for its node (a table indexed by the node's low bits: two nodes that meet there count as one, which
                // only shortens the batch), the highest key keeps it, among equal keys the lowest job.
#pragma unroll
                for (int u = 0; u < 2; ++u) if (usable[u]) atomicMax(&claim_k[s_node[u] & (CLAIMS - 1)], key_[u]);
                __syncwarp();
#pragma unroll
                for (int u = 0; u < 2; ++u) if (usable[u] && claim_k[s_node[u] & (CLAIMS - 1)] == key_[u]) atomicMin(&claim_j[s_node[u] & (CLAIMS - 1)], j_[u]);
                __syncwarp();
                bool lower[2];
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    lower[u] = usable[u] && !(claim_k[s_node[u] & (CLAIMS - 1)] == key_[u] && claim_j[s_node[u] & (CLAIMS - 1)] == j_[u]);
                __syncwarp();
#pragma unroll
                for (int u = 0; u < 2; ++u) if (usable[u]) { claim_k[s_node[u] & (CLAIMS - 1)] = 0u; claim_j[s_node[u] & (CLAIMS - 1)] = 0x7fffffff; }
                const uint32_t t_node = __reduce_max_sync(FULL, max(lower[0] ? key_[0] : 0u, lower[1] ? key_[1] : 0u));
                if (t_node > t) t = t_node;
                const uint32_t t_bound = __reduce_max_sync(FULL, max(usable[0] && key_[0] > t ? (s_bound[0] < key_[0] ? s_bound[0] : key_[0]) : 0u,
                                                                      usable[1] && key_[1] > t ? (s_bound[1] < key_[1] ? s_bound[1] : key_[1]) : 0u));
                if (t_bound > t) t = t_bound;
                unsigned acc[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) acc[u] = __ballot_sync(FULL, usable[u] && key_[u] > t);
                n_acc = __popc(acc[0]) + __popc(acc[1]);
                int my_order[2] = { 0, 0 };                  // position among the taken ones (the step log wants it)
                if (n_acc > room || A.step_log) {
                    __syncwarp();
#pragma unroll
                    for (int x = 0; x < 2; ++x)
                        for (unsigned m = acc[x]; m; m &= m - 1) {
                            const u64 o = sh.sel[__ffs(m) - 1 + 32 * x];
                            my_order[0] += int(o > mine[0]); my_order[1] += int(o > mine[1]);
                        }
                    if (n_acc > room) {
#pragma unroll
                        for (int u = 0; u < 2; ++u) acc[u] = __ballot_sync(FULL, ((acc[u] >> lane) & 1u) && my_order[u] < room);
                        n_acc = room;
                    }
                }
                // warp 1 stores what the second candidates change, this warp the first ones' (different nodes, different slots)
                BatchOut o0;
                o0.elig = elig[0]; o0.ok = s_ok[0]; o0.maxc = s_maxc[0]; o0.multi = s_multi[0];
                o0.slot = s_slot[0]; o0.node = s_node[0]; o0.type = s_type[0]; o0.dgc = s_dgc[0]; o0.k = s_k[0]; o0.dm = s_dm[0]; o0.bound = 0u;
                const bool taken0 = (acc[0] >> lane) & 1u;
                const bool md0 = __any_sync(FULL, taken0 && o0.ok && o0.maxc);
                sh.order_b[lane] = my_order[1];
                if (lane == 0) {
                    sh.acc_b = acc[1]; sh.steps0_b = steps0;
                    if (n_acc > 0) { sh.steps = steps0 + n_acc; sh.maxc_dirty = md0 ? 1 : 0; }
                }
                pair_barrier(3);
                batch_apply(sp, v, sh, A.hc, A.tr, A.step_log, N, bst + 3 * lane, taken0, o0, j_[0], steps0 + my_order[0], lane);
            }
            // ---- a chain of general commits ------------------------------------------------------------------
            // Whatever the top candidate needs (a migration, growth onto whole nodes, the first placement of an
            // unallocated job), its commit is worked out by the whole warp on the real cluster state, and so is
            // every candidate after it for which the order of the sequential rule can be proved: all offered
            // candidates and the first entries of the best class are fetched in one wave of loads and staged in
            // shared memory in the rule's order (key, then lowest job); the next one is committed while its key
            // exceeds every key that was not offered (M), every new candidate of the jobs committed before it in
            // this turn and, once a commit has given resources back, every increment that had no place before
            // (it might have one now).  A candidate whose own increment changed under the commits before it
            // ends the chain, and so does a class that lost its place.
            // Each lane prepares its candidate for the usual commit -- a job on one node whose target's curve entry
            // is usable as it stands: what it holds and wants as node words, the memory of both, the slot it will
            // have afterwards -- so that such a commit only has to find the node, compare the memory and store.
            // Everything else (whole nodes, an entry that needs the table, too little memory) goes through commit_warp.
            if (go && n_acc == 0) {
                uint32_t M = __reduce_max_sync(FULL, lane < 16 ? sh.red_key2[OFFER * lane] : 0u);
                const uint32_t Mblk = __reduce_max_sync(FULL, lane < 16 ? sh.red_key2[OFFER * lane + 1] : 0u);
                // -- stage the offered candidates of running jobs
                bool is_slot[2]; u64 mine[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    is_slot[u] = lane + 32 * u < CLS_G && key_[u] != 0u;
                    mine[u] = is_slot[u] ? ((u64(key_[u]) << 32) | (u64(uint32_t(KEY_JOB_MASK) - uint32_t(j_[u])) << 6) | u64(63 - lane - 32 * u)) : 0ull;
                    sh.sel[lane + 32 * u] = mine[u];
                }
                __syncwarp();
                const int n_all = __popc(__ballot_sync(FULL, is_slot[0])) + __popc(__ballot_sync(FULL, is_slot[1]));
                // the 32 best are staged, one a lane; the key of the next one bounds the chain like the keys that were not offered
                const int n_sc = min(n_all, 32);
                int rank[2] = { 0, 0 };
                {
                    const ulonglong2 *sel2 = reinterpret_cast<const ulonglong2 *>(sh.sel);
#pragma unroll 6
                    for (int i = 0; i < CLS_G / 2; ++i) {
                        const ulonglong2 o = sel2[i];
                        rank[0] += int(o.x > mine[0]) + int(o.y > mine[0]);
                        rank[1] += int(o.x > mine[1]) + int(o.y > mine[1]);
                    }
                }
                unsigned char *perm = reinterpret_cast<unsigned char *>(bres);          // rank -> candidate (the words of a batch's hand-over are idle here)
#pragma unroll
                for (int u = 0; u < 2; ++u) if (is_slot[u]) perm[rank[u]] = (unsigned char)(lane + 32 * u);
                __syncwarp();
                if (n_all > 32) M = max(M, sh.red_key[perm[32]]);
                {
                    if (lane < n_sc) {
                        const int cidx = perm[lane];
                        const uint32_t key = sh.red_key[cidx]; const int my_j = sh.red_j[cidx];
                        const int s = int(sh.red_pay[cidx]);
                        const int u = 0;
                        const SlotA a = v.sa[s];
                        const int type_gpu = int(key >> 31);
                        const int gi = pk_gi(a.packed), ci = pk_ci(a.packed);
                        const int gi2 = type_gpu ? pk_next_gi(a.packed) : gi, ci2 = type_gpu ? ci : ci + 1;
                        const size_t o = hc_idx(sp, my_j, gi2, ci2);
                        ChainRec &r = chain[lane + u];
                        const int4 b4 = *reinterpret_cast<const int4 *>(v.sb + s);
                        const int4 c4 = *reinterpret_cast<const int4 *>(A.hc + o);
                        const int4 t_lo = reinterpret_cast<const int4 *>(A.tr + o)[0];
                        r.nq = reinterpret_cast<const int4 *>(A.tr + o)[1];
                        const int g = v.gl[gi], c = v.clv[ci], g2 = v.gl[gi2], c2 = v.clv[ci2];
                        const bool f_ok = c4.z >= 0 && c4.z < sp.nM;
                        const bool cand_ok = c4.y >= 0 && c4.y < sp.P && f_ok && __int_as_float(c4.x) > 0.0f && c4.w != 0
                                             && __int_as_float(c4.x) > __int_as_float(b4.x);
                        const bool lean = cand_ok && g <= sp.Gn && g2 <= sp.Gn;
                        const bool fz_g = pk_fz_g(a.packed), fz_c = pk_fz_c(a.packed);
                        r.b = b4; r.cand = c4; r.t_lo = t_lo;
                        r.cur = make_int4((g << 16) | c, (g2 << 16) | c2, a.node, 0);
                        r.mem = make_longlong2(v.ml[b4.z], f_ok ? v.ml[c4.z] : 0);
                        r.na = make_int4(fz_g ? 0 : t_lo.x, fz_c ? 0 : t_lo.y, int(pack(gi2, ci2, t_lo.z, fz_g, fz_c)), -1);
                        r.nb = make_int4(c4.x, c4.y, c4.z, b4.w);
                        r.m = make_int4(int(key), my_j, s, gi2 | (ci2 << 8) | (type_gpu << 16) | (int(lean) << 17));
                    }
                }
                // -- and the first entries of the best class of unallocated jobs (its head is the candidate of lane CLS_G)
                const uint32_t cls_key = __shfl_sync(FULL, key_[1], CLS_G - 32), cls_pay = __shfl_sync(FULL, pay_[1], CLS_G - 32);
                int n_ce = 0, cls_t = -1, cls_ptr0 = 0, cls_end0 = 0;
                u64 ce_k = 0ull; float ce_w = 0.0f;          // lane i: key and weight of entry i of the class (i <= CHAIN_CLS)
                if (cls_key != 0u) {
                    cls_t = int(cls_pay & 0x7fffffffu);
                    const int gi2 = cls_t / sp.nC, ci2 = cls_t - gi2 * sp.nC;
                    cls_ptr0 = v.cls_ptr[cls_t]; cls_end0 = v.cls_end[cls_t];
                    n_ce = min(cls_end0 - cls_ptr0, CHAIN_CLS);
                    const int idx = cls_ptr0 + lane;
                    if (lane <= CHAIN_CLS && idx < cls_end0) { ce_k = A.keys[idx]; ce_w = A.sorted_w[idx]; }
                    if (lane < n_ce) {
                        const int j = key_job(ce_k);
                        const size_t o = hc_idx(sp, j, gi2, ci2);
                        ChainRec &r = chain[CHAIN_SLOTS + lane];
                        const int4 c4 = *reinterpret_cast<const int4 *>(A.hc + o);
                        const int4 t_lo = reinterpret_cast<const int4 *>(A.tr + o)[0];
                        r.nq = reinterpret_cast<const int4 *>(A.tr + o)[1];
                        const int g2 = v.gl[gi2], c2 = v.clv[ci2];
                        const bool f_ok = c4.z >= 0 && c4.z < sp.nM;
                        const bool lean = c4.y >= 0 && c4.y < sp.P && f_ok && __int_as_float(c4.x) > 0.0f && c4.w != 0 && g2 <= sp.Gn;
                        r.b = make_int4(0, -1, 0, __float_as_int(ce_w));
                        r.cand = c4; r.t_lo = t_lo;
                        r.cur = make_int4(0, (g2 << 16) | c2, -1, 0);
                        r.mem = make_longlong2(0, f_ok ? v.ml[c4.z] : 0);
                        r.na = make_int4(t_lo.x, t_lo.y, int(pack(gi2, ci2, t_lo.z, false, false)), -1);
                        r.nb = make_int4(c4.x, c4.y, c4.z, __float_as_int(ce_w));
                        r.m = make_int4(int(0x80000000u | key_gain_bits(ce_k)), j, -1, gi2 | (ci2 << 8) | (1 << 16) | (int(lean) << 17));
                    }
                }
                const uint32_t ce_key32 = ce_k ? (0x80000000u | key_gain_bits(ce_k)) : 0u;
                __syncwarp();

                int i_s = 0, i_c = 0, done = 0;
                // counters of the block, the same on every lane; shared memory follows every change
                int ne = sh.n_empty, n_sl = sh.n_slots, e_lo = sh.empty_lo, ver_r = sh.ver;
                // while an empty node remains and every maxc[] entry is the node's core count no commit on single nodes changes maxc[]
                bool all_max = __all_sync(FULL, lane >= sp.n_small || v.maxc[lane] == sp.Cn);
                const int gl_l = lane < sp.n_small ? v.gl[lane] : 0x7fff;      // lane i answers for GPU level i when maxc[] is checked
                uint32_t b_new = 0u, b_blk = 0u;       // new candidates of the jobs committed in this turn: with / without a place
                bool freed = false, last_cls_ok = false;
                bool cls_open = true;                  // entries of the class are taken until one of them is rejected: a run of
                                                       // rejections is settled faster by the turn that looks for one
                while (done < room) {
                    const bool c_avail = cls_open && i_c < n_ce;
                    const int4 ms = i_s < n_sc ? chain[i_s].m : make_int4(0, 0x7fffffff, 0, 0);
                    const int4 mc = c_avail ? chain[CHAIN_SLOTS + i_c].m : make_int4(0, 0x7fffffff, 0, 0);
                    const bool take_c = uint32_t(mc.x) > uint32_t(ms.x) || (mc.x == ms.x && mc.y < ms.y);
                    const int4 mx = take_c ? mc : ms;
                    const uint32_t kx = uint32_t(mx.x);
                    if (kx == 0u) break;
                    if (done > 0) {
                        uint32_t T = max(M, b_new);
                        if (freed) T = max(T, max(Mblk, b_blk));
                        // the class's next entry when it is not among the stream heads (not staged, or held back)
                        if (!c_avail) T = max(T, __shfl_sync(FULL, ce_key32, i_c & 31));
                        if (!(kx > T)) break;
                    }
                    const ChainRec *r = &chain[take_c ? CHAIN_SLOTS + i_c : i_s];
                    const int j = mx.y, gi2 = mx.w & 0xff, ci2 = (mx.w >> 8) & 0xff, type_gpu = (mx.w >> 16) & 1;
                    const bool lean = (mx.w >> 17) & 1;
                    // everything the usual commit reads of the record, in one wave
                    const int4 cur = r->cur;
                    const longlong2 mm = r->mem;            // x = memory held, y = memory of the target's entry
                    const int4 na4 = r->na, nq4 = r->nq;
                    const int need_old = cur.x, need_new = cur.y, node = cur.z;
                    const int g2 = need_new >> 16, c2 = need_new & 0xffff;
                    const int s = take_c ? n_sl : mx.z;
                    const int w_n = node >= 0 ? v.gc[node] : 0;
                    const int64_t fm_n = node >= 0 ? v.free_m[node] : 0;
                    const int mx_t = g2 <= sp.Gn ? v.maxc[gi2] : -1;
                    SlotA na; SlotC nq;
                    na.gain_g = __int_as_float(na4.x); na.gain_c = __int_as_float(na4.y); na.packed = uint32_t(na4.z); na.node = -1;
                    nq = *reinterpret_cast<const SlotC *>(&nq4);
                    if (done > 0 && !lean) {             // (the usual commit sees by itself whether its increment still has a place)
                        if (take_c) {                    // has the class still got a place?
                            bool has;
                            if (g2 <= sp.Gn) has = mx_t >= c2;
                            else { const int k2 = g2 >> sp.log2Gn; has = (c2 + k2 - 1) / k2 <= sp.Cn && ne >= k2; }
                            if (!has) break;
                        } else {                         // is this still the job's best increment that has a place?
                            uint32_t kg, kc, blk;
                            slot_keys(sp, v, ne, v.sa[s], v.sc[s], w_n, kg, kc, blk);
                            if ((kg ? kg : kc) != kx) break;
                        }
                    }
                    bool ok = false, settled = false;
                    int w_new_t = 0;
                    if (lean) {
                        const int d = need_new - need_old;          // (extra GPUs << 16) + extra cores: neither is negative
                        const bool stay = node >= 0 && fg_of(w_n) >= (d >> 16) && fc_of(w_n) >= (d & 0xffff);
                        const bool has = stay || mx_t >= c2;
                        // The commits before it may have taken the place this increment had.  (An increment of the job that
                        // had no place can only have got one after resources were given back, and then its key is among
                        // those the candidate had to exceed.)
                        if (!has && done > 0) break;
                        const int target = stay ? node : (has ? first_fit_warp(v, g2, c2, lane) : -1);
                        if (target >= 0) {
                            const int w_t = stay ? w_n : v.gc[target];
                            const int64_t fm = stay ? fm_n + mm.x : v.free_m[target];
                            const int mxc = lane < sp.n_small ? v.maxc[lane] : -1;
                            if (mm.y <= fm) {
                                // the highest memory level that fits the node is at or above the plan's own: the entry stands
                                const bool moved = node >= 0 && !stay;
                                const int w_new_n = w_n + need_old;
                                w_new_t = w_t - (stay ? d : need_new);
                                const int ne0 = ne;
                                if (moved) {
                                    v.gc[node] = w_new_n; v.free_m[node] = fm_n + mm.x;
                                    if (fg_of(w_new_n) == sp.Gn) { ++ne; if (node < e_lo) { e_lo = node; sh.empty_lo = node; } }
                                }
                                v.gc[target] = w_new_t; v.free_m[target] = fm - mm.y;
                                if (!stay && fg_of(w_t) == sp.Gn) --ne;
                                // can maxc[] have changed?
                                bool ch;
                                if (ne > 0) ch = !all_max;          // (then every entry is the node's core count)
                                else {
                                    const int ot = fg_of(w_t) >= gl_l ? fc_of(w_t) : -1, nt = fg_of(w_new_t) >= gl_l ? fc_of(w_new_t) : -1;
                                    bool c1 = (ot == mxc && nt < ot) || nt > mxc;
                                    if (moved) {
                                        const int on = fg_of(w_n) >= gl_l ? fc_of(w_n) : -1, nn = fg_of(w_new_n) >= gl_l ? fc_of(w_new_n) : -1;
                                        c1 = c1 || (on == mxc && nn < on) || nn > mxc;
                                    }
                                    ch = __any_sync(FULL, c1);
                                }
                                bool changed = false;
                                if (ch) {
                                    __syncwarp();
                                    changed = rebuild_maxc_changed(sp, v, lane);
                                    all_max = __all_sync(FULL, lane >= sp.n_small || v.maxc[lane] == sp.Cn);
                                }
                                if (ne != ne0) sh.n_empty = ne;
                                if (ne != ne0 || changed) { ++ver_r; sh.ver = ver_r; }
                                na.node = target;
                                if (take_c) { ++n_sl; sh.n_slots = n_sl; }
                                if (lane == 0) {
                                    if (moved) atomicOr(&v.tb[node >> 5], 1u << (node & 31));
                                    atomicOr(&v.tb[target >> 5], 1u << (target & 31));
                                    v.sa[s] = na; *reinterpret_cast<int4 *>(v.sb + s) = r->nb; v.sc[s] = nq;
                                    if (take_c) v.sj[s] = j;
                                    sh.dirty[dirty_of(s)] = 1;
                                    if (A.step_log) A.step_log[steps0 + done] = (j << 2) | ((type_gpu ? 0 : 1) << 1) | 1;
                                }
                                freed = freed || moved;
                                ok = true; settled = true;
                            }
                        }
                    }
                    if (!settled) {
                        const int4 rc = r->cand, t_lo = r->t_lo;
                        HotCurve cand; cand.val = __int_as_float(rc.x); cand.plan = rc.y; cand.f = rc.z; cand.ok = rc.w;
                        const int4 rb = r->b;
                        SlotA a0; a0.gain_g = a0.gain_c = 0.0f; a0.packed = 0u; a0.node = node;
                        if (!take_c) a0 = v.sa[s];                  // (its slot is as it was when the turn began)
                        SlotB nb; nb.val = __int_as_float(rb.x); nb.plan = rb.y; nb.f_level = rb.z; nb.w = __int_as_float(rb.w);
                        bool fz_g = pk_fz_g(a0.packed), fz_c = pk_fz_c(a0.packed);
                        Committed cm;
                        __syncwarp();
                        if (take_c) ok = commit_warp<false, COMMIT_CHAIN>(sp, v, sh, A.cv, A.cp, A.cg, A.feas, j, -1, 0, -1, 0.0f, 0, gi2, ci2, cand, true, lane, cm);
                        else ok = commit_warp<true, COMMIT_CHAIN>(sp, v, sh, A.cv, A.cp, A.cg, A.feas, j, pk_gi(a0.packed), pk_ci(a0.packed), node,
                                                                  nb.val, nb.f_level, gi2, ci2, cand, true, lane, cm);
                        __syncwarp();
                        ne = sh.n_empty; e_lo = sh.empty_lo; ver_r = sh.ver;
                        all_max = __all_sync(FULL, lane >= sp.n_small || v.maxc[lane] == sp.Cn);
                        if (ok) {
                            // committed with the curve's own value (the usual case): the transition record has the rest
                            const bool rec = cm.plan == cand.plan && cm.val == cand.val;
                            int ng_ = t_lo.z, nc_ = t_lo.w; float gg = __int_as_float(t_lo.x), gc = __int_as_float(t_lo.y);
                            if (!rec) {
                                const int lvl = gi2 + 1 + lane;
                                const float v_lane = lvl < sp.nG ? A.hc[hc_idx(sp, j, lvl, ci2)].val : 0.0f;
                                const float vc = ci2 + 1 < sp.nC ? A.hc[hc_idx(sp, j, gi2, ci2 + 1)].val : 0.0f;
                                gains_from_column(sp, nb.w, gi2, ci2, cm.val, v_lane, vc, lane, ng_, gg, nc_, gc);
                                nq = make_slotc(sp, v.gl, v.clv, gi2, ci2, ng_, nc_);
                            }
                            na.gain_g = fz_g ? 0.0f : gg; na.gain_c = fz_c ? 0.0f : gc;
                            na.packed = pack(gi2, ci2, ng_, fz_g, fz_c); na.node = cm.first;
                            nb.val = cm.val; nb.plan = cm.plan; nb.f_level = cm.f;
                            if (lane == 0) {
                                v.sa[s] = na; v.sb[s] = nb; v.sc[s] = nq;
                                if (take_c) v.sj[s] = j;
                                sh.dirty[dirty_of(s)] = 1;
                            }
                            if (take_c) { ++n_sl; sh.n_slots = n_sl; }
                            w_new_t = v.gc[na.node];
                            freed = freed || cm.freed != 0;
                        } else if (!take_c) {
                            // rejected: the (job, type) pair is frozen, the other increment stays as it is
                            if (type_gpu) { fz_g = true; a0.gain_g = 0.0f; } else { fz_c = true; a0.gain_c = 0.0f; }
                            a0.packed = pack(pk_gi(a0.packed), pk_ci(a0.packed), pk_next_gi(a0.packed), fz_g, fz_c);
                            if (lane == 0) { v.sa[s] = a0; sh.dirty[dirty_of(s)] = 1; }
                        }
                        if (lane == 0 && A.step_log) A.step_log[steps0 + done] = (j << 2) | ((type_gpu ? 0 : 1) << 1) | int(ok);
                    }
                    if (ok) {
                        // what the job wants next, for the candidates after it in this turn
                        uint32_t kp, blk;
                        slot_keys_uniform(sp, v, ne, na, nq, w_new_t, kp, blk);
                        b_new = max(b_new, kp); b_blk = max(b_blk, blk);

                    }
                    if (take_c) { last_cls_ok = ok; if (!ok) cls_open = false; ++i_c; } else ++i_s;
                    ++done;
                }
                // the class moves on past the entries used (consumed whether or not their commits succeeded)
                const u64 nk = __shfl_sync(FULL, ce_k, i_c & 31);
                const float nw = __shfl_sync(FULL, ce_w, i_c & 31);
                if (lane == 0) {
                    if (i_c > 0) {
                        const int np = cls_ptr0 + i_c;
                        v.cls_ptr[cls_t] = np; v.cls_top[cls_t] = np < cls_end0 ? nk : 0ull; v.cls_w[cls_t] = np < cls_end0 ? nw : 0.0f;
                        sh.dirty[CLS_G] = 1;
                        if (last_cls_ok) cls_went[cls_t >> 5] |= 1u << (cls_t & 31); else cls_went[cls_t >> 5] &= ~(1u << (cls_t & 31));
                    }
                    sh.steps = steps0 + done;
                }
                n_acc = done;
            }
            if (lane == 0) sh.stop = (go && n_acc > 0) ? 0 : 1;      // a turn always settles at least one step
        } else if (warp == 1) {
            // the second candidate of every lane of warp 0 when the turn is a batch
            pair_barrier(1);
            if (sh.batch_go) {
                const unsigned FULL = 0xffffffffu;
                const int n_empty = sh.n_empty;
                const bool saturated = n_empty > 0 && __all_sync(FULL, lane >= sp.n_small || v.maxc[lane] == sp.Cn);
                int mx_r[4], gl_r[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) { mx_r[u] = u < sp.n_small ? v.maxc[u] : -2; gl_r[u] = u < sp.n_small ? v.gl[u] : 0x7fffffff; }
                BatchOut o;
                batch_candidate(sp, v, A.hc, A.tr, n_empty, saturated, mx_r, gl_r, sh.red_key[lane + 32], sh.red_pay[lane + 32], sh.red_j[lane + 32],
                                bst + 3 * (lane + 32), o);
                bres[2 * lane] = make_int4(int(o.elig) | (int(o.ok) << 1) | (int(o.maxc) << 2) | (int(o.multi) << 3) | (o.type << 4), o.slot, o.node, o.dgc);
                bres[2 * lane + 1] = make_int4(o.k, int(o.bound), int(uint32_t(o.dm)), int(uint32_t(uint64_t(o.dm) >> 32)));
                pair_barrier(2);
                pair_barrier(3);                     // warp 0 has decided which candidates are taken
                const bool taken = (sh.acc_b >> lane) & 1u;
                const bool md = batch_apply(sp, v, sh, A.hc, A.tr, A.step_log, N, bst + 3 * (lane + 32), taken, o, sh.red_j[lane + 32],
                                            sh.steps0_b + sh.order_b[lane], lane);
                if (md && lane == 0) sh.maxc_dirty = 1;
            }
        }
        __syncthreads();
        if (sh.stop) break;
    }

    // ---- results -----------------------------------------------------------------------------------------
    for (int s = tid; s < sh.n_slots; s += RT) {
        const SlotA a = v.sa[s]; const SlotB b = v.sb[s];
        rubick_assignment r;
        r.g = sp.g_levels[pk_gi(a.packed)]; r.c = sp.c_levels[pk_ci(a.packed)]; r.m_bytes = sp.m_levels[b.f_level];
        r.plan = b.plan; r.first_node = a.node; r.n_nodes = max(r.g >> sp.log2Gn, 1);
        r.thr = b.val; r.status = RUBICK_RUNNING; r.m_level = b.f_level;
        A.out[v.sj[s]] = r;
    }
    if (A.node_out)
        for (int n = tid; n < N; n += RT) {
            rubick_node nd;
            nd.free_g = fg_of(v.gc[n]); nd.free_c = fc_of(v.gc[n]); nd.free_m = v.free_m[n]; nd.owner = v.owner[n]; nd.reserved = 0;
            A.node_out[n] = nd;
        }
    if (tid == 0) {
        *A.steps_out = sh.steps;
        if (sh.capped) atomicOr(A.status, DS_STEP_CAP);
    }
}

// ---- host side ------------------------------------------------------------------------------------------
struct Layout {
    int n_pad, slot_cap, slots_in_smem;
    size_t smem, off_hc, off_tr, off_keys, off_w, off_pa, off_glist, off_isg, off_sa, off_sb, off_sc, off_sj, total;
};

static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

static size_t fixed_smem(const Space &sp, int N)
{
    const size_t n_cls = size_t(sp.nG) * sp.nC;
    const size_t n_pad = (size_t(N) + 127) & ~size_t(127);
    const size_t fixed = n_pad * 4 + size_t(N) * 12 + n_cls * 24 + size_t(2 * RUBICK_MAX_G_LEVELS + RUBICK_MAX_C_LEVELS) * 4
                         + size_t(RUBICK_MAX_M_LEVELS) * 8 + n_pad / 8;
    return (fixed + 15) & ~size_t(15);
}

static Layout make_layout(const Space &sp, int J, int N)
{
    Layout L;
    int n = 2;
    while (n < J) n <<= 1;
    L.n_pad = n;
    const long long gpus = (long long)N * sp.Gn;
    L.slot_cap = int(gpus < J ? gpus : J);
    if (L.slot_cap < 1) L.slot_cap = 1;
    const size_t fixed = fixed_smem(sp, N);
    const size_t slots = size_t(L.slot_cap) * SLOT_BYTES;
    L.slots_in_smem = fixed + slots <= SMEM_LIMIT;
    L.smem = fixed + (L.slots_in_smem ? slots : 0);
    const size_t gs = L.slots_in_smem ? 0 : size_t(L.slot_cap);
    size_t o = 0;
    L.off_hc = o; o = align256(o + size_t(J) * sp.nG * sp.nC * sizeof(HotCurve));
    L.off_tr = o; o = align256(o + size_t(J) * sp.nG * sp.nC * sizeof(Trans));
    L.off_keys = o; o = align256(o + size_t(n) * 8);
    L.off_w = o; o = align256(o + size_t(n) * 4);
    L.off_pa = o; o = align256(o + size_t(J) * sizeof(PhaseA));
    L.off_glist = o; o = align256(o + size_t(J) * 4);
    L.off_isg = o; o = align256(o + size_t(J) * 4);
    L.off_sa = o; o = align256(o + gs * sizeof(SlotA));
    L.off_sb = o; o = align256(o + size_t(L.slot_cap) * sizeof(SlotB));
    L.off_sc = o; o = align256(o + gs * sizeof(SlotC));
    L.off_sj = o; o = align256(o + gs * 4);
    L.total = o;
    return L;
}

}  // namespace fastround

bool round_fast_supported(const Space &sp, int J, int N)
{
    using namespace fastround;
    if (J < 1 || J >= (1 << KEY_JOB_BITS)) return false;
    // node words and slot requirements hold 15 / 16-bit fields
    if (sp.Cn > 32767 || sp.Gn > 16384 || sp.g_levels[sp.nG - 1] > 32767 || sp.c_levels[sp.nC - 1] > 32767) return false;
    if (size_t(sp.nG) * sp.nC > 65535) return false;
    return fixed_smem(sp, N) <= SMEM_LIMIT;
}

size_t round_fast_scratch_need(const Space &sp, int J, int N)
{
    return fastround::make_layout(sp, J, N).total;
}

cudaError_t launch_round_fast(const Space &sp, const rubick_job *d_jobs, int J, const float *d_cv, const int32_t *d_cp,
                              const int32_t *d_cg, const uint32_t *d_feas, int N, int max_steps,
                              rubick_assignment *d_out, rubick_node *d_node_out, int32_t *d_step_log,
                              void *d_scratch, const int32_t *d_quota, int n_tenants,
                              uint32_t *d_status, int32_t *d_steps, cudaStream_t st, const int4 *d_top)
{
    using namespace fastround;
    const Layout L = make_layout(sp, J, N);
    unsigned char *base = static_cast<unsigned char *>(d_scratch);
    HotCurve *hc = reinterpret_cast<HotCurve *>(base + L.off_hc);
    u64 *keys = reinterpret_cast<u64 *>(base + L.off_keys);
    float *sw = reinterpret_cast<float *>(base + L.off_w);
    PhaseA *pa = reinterpret_cast<PhaseA *>(base + L.off_pa);

    const long long natural = (long long)J * (sp.nG + sp.nC + 2) + 1;
    if ((long long)max_steps > natural) max_steps = int(natural < 0x7fffffffLL ? natural : 0x7fffffffLL);

    Trans *tr = reinterpret_cast<Trans *>(base + L.off_tr);
    round_prepare_kernel<<<J, 256, 0, st>>>(sp, d_jobs, d_cv, d_cp, d_cg, d_feas, hc, tr, d_top); count_launch();
    round_keys_kernel<<<(L.n_pad + 127) / 128, 128, 0, st>>>(sp, d_jobs, J, hc, d_cp, d_cg, keys, L.n_pad, pa, d_out,
                                                                reinterpret_cast<int32_t *>(base + L.off_isg)); count_launch();
    {
        const int n = L.n_pad, tile = n < SORT_TILE ? n : SORT_TILE;
        bool sorted = false;
        if (n > SORT_TILE && n <= SORT_TILE * SORT_CLUSTER_MAX) {
            // two to eight tiles: one cluster sorts them in one launch
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(unsigned(n / SORT_TILE)); cfg.blockDim = dim3(SORT_T); cfg.dynamicSmemBytes = 0; cfg.stream = st;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = unsigned(n / SORT_TILE); at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            cfg.attrs = at; cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, round_sort_cluster_kernel, keys, n, d_jobs, sw) == cudaSuccess) { count_launch(); sorted = true; }
            else (void)cudaGetLastError();      // a device that cannot place the cluster: the launches below do the same work
        }
        if (!sorted) {
            // every stage up to the tile size, tile by tile; then stage by stage: wide strides in global memory, the rest in tiles
            round_sort_tile_kernel<<<n / tile, SORT_T, 0, st>>>(keys, n, tile, 2, tile, n == tile, d_jobs, sw); count_launch();
            for (int k = tile << 1; k <= n; k <<= 1) {
                for (int s = k >> 1; s >= tile; s >>= 1) {
                    round_sort_pass_kernel<<<((n >> 1) + 255) / 256, 256, 0, st>>>(keys, n, k, s);
                    count_launch();
                }
                round_sort_tile_kernel<<<n / tile, SORT_T, 0, st>>>(keys, n, tile, k, k, k == n, d_jobs, sw); count_launch();
            }
        }
    }
    cudaError_t e;

    RoundArgs A;
    A.jobs = d_jobs; A.J = J; A.cv = d_cv; A.cp = d_cp; A.cg = d_cg; A.feas = d_feas; A.N = N; A.max_steps = max_steps;
    A.out = d_out; A.node_out = d_node_out; A.step_log = d_step_log;
    A.hc = hc; A.tr = tr; A.keys = keys; A.sorted_w = sw; A.n_pad = L.n_pad; A.pa = pa;
    A.glist = reinterpret_cast<int32_t *>(base + L.off_glist);
    A.is_guar = reinterpret_cast<const int32_t *>(base + L.off_isg);
    A.sa_g = reinterpret_cast<SlotA *>(base + L.off_sa); A.sb_g = reinterpret_cast<SlotB *>(base + L.off_sb);
    A.sc_g = reinterpret_cast<SlotC *>(base + L.off_sc); A.sj_g = reinterpret_cast<int32_t *>(base + L.off_sj);
    A.slots_in_smem = L.slots_in_smem; A.slot_cap = L.slot_cap;
    A.quota = d_quota; A.n_tenants = n_tenants;
    A.status = d_status; A.steps_out = d_steps;
    e = cudaFuncSetAttribute(greedy_round_fast_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(SMEM_LIMIT));
    if (e != cudaSuccess) return e;
    greedy_round_fast_kernel<<<1, RT, L.smem, st>>>(sp, A); count_launch();
    return cudaGetLastError();
}

}  // namespace rubick
