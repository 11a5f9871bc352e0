// Best plan per (job, GPU level, CPU level, host-memory level) and the resource-sensitivity
// curve (paper Section 5.2): an argmax over the plans of one GPU level that are feasible at a
// memory level, lowest plan index on ties, then the running maximum along the GPU axis.
//
// Two kernels.  Feasibility words are thresholds in the memory level, so a plan is described by its
// first feasible level f.  Under the memory rule of this library the host-memory need of a plan
// depends only on its GPU count and on whether it offloads, so within one GPU level all feasible
// plans without offload share one f and all feasible plans with offload share another: two
// "classes" per level (even / odd plan indices).
//
// best_plan_kernel streams the table for jobs of that shape.  One CTA per job; the mask words become
// one float per plan in shared memory (1 = feasible somewhere) and one first level per (GPU level,
// class).  A warp takes BEST_ROWS core levels at a time and walks the row in plan order, 32 quads
// per step with 16-byte loads issued BEST_STAGES steps ahead; every lane keeps the running
// (value, index) maximum of both classes for its own quads (a strict "greater" keeps the lowest
// index, infeasible plans are multiplied by 0 and never win).  Where a GPU level ends inside a step
// the lanes below the boundary are taken first; two warp reductions per class (maximum of the value
// bits, then minimum index among the lanes that hold it) finish the level, lane m combines the two
// classes for memory level m (a class counts when its first level is <= m), folds the result into
// the running maximum along the GPU axis and stores its outputs.  No shared-memory buckets, no
// atomics, no separate epilogue: loads stay in flight while results are written.
//
// A job whose mask does not have that shape (any caller may pass scattered thresholds) is appended
// to a to-do list and handled by best_plan_scattered_kernel, which makes no assumption: 16-bit
// "slots" (GPU level * 32 + first level) per plan, per-lane runs flushed into per-warp buckets with
// a 64-bit shared-memory max on (value bits << 32 | ~index), then a maximum over the occupied
// buckets at or below each memory level.
//
// The table is read once (4 bytes per candidate); outputs are 12 bytes per (g, c, m).

#include "rubick_internal.cuh"

namespace rubick {

constexpr int BEST_WARPS = 12;        // at most; fewer when core levels are few (or, scattered kernel, buckets would not fit)
constexpr int BEST_ROWS = 2;          // CPU levels a warp processes together
constexpr int BEST_STAGES = 3;        // steps of 32 quads a warp has in flight per row
constexpr int BEST_UNROLL = 2;        // scattered kernel: quads per lane in flight per row
constexpr unsigned FULL = 0xffffffffu;
constexpr int NO_LEVEL = 255;         // first level of a class without feasible plans

struct Best {
    float ev[BEST_ROWS], ov[BEST_ROWS];     // running maxima of the even (no offload) / odd (offload) class per row
    int ei[BEST_ROWS], oi[BEST_ROWS];       // their plan indices
};

__device__ __forceinline__ void take(float &bv, int &bi, float v, int i, bool on)
{
    const bool up = on && v > bv;
    bv = up ? v : bv;
    bi = up ? i : bi;
}

// lanes with `on` fold the four plans of quad q into their running maxima
__device__ __forceinline__ void accumulate(Best &b, const float4 (&v)[BEST_ROWS], int q, bool on)
{
#pragma unroll
    for (int k = 0; k < BEST_ROWS; ++k) {
        take(b.ev[k], b.ei[k], v[k].x, 4 * q, on);
        take(b.ov[k], b.oi[k], v[k].y, 4 * q + 1, on);
        take(b.ev[k], b.ei[k], v[k].z, 4 * q + 2, on);
        take(b.ov[k], b.oi[k], v[k].w, 4 * q + 3, on);
    }
}

__device__ __forceinline__ float4 mul4(float4 a, float4 m) { return make_float4(a.x * m.x, a.y * m.y, a.z * m.z, a.w * m.w); }

__global__ void __launch_bounds__(BEST_WARPS * 32, 3)
best_plan_kernel(const __grid_constant__ Space sp, const float *__restrict__ thr, const uint32_t *__restrict__ feas,
                 int J, unsigned flags, float *__restrict__ best_val, int32_t *__restrict__ best_plan,
                 int32_t *__restrict__ best_g, uint32_t *__restrict__ status, int32_t *__restrict__ todo)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float4 *maskf = reinterpret_cast<float4 *>(smem_raw);                 // [Q rounded up to 32] 1 = the plan is feasible at some level
    __shared__ int s_lo[2 * RUBICK_MAX_G_LEVELS], s_hi[2 * RUBICK_MAX_G_LEVELS];   // lowest / highest first level per (level, class)

    const int j = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const uint32_t full = sp.nM >= 32 ? FULL : ((1u << sp.nM) - 1u);
    const int n_pairs = (sp.nC + BEST_ROWS - 1) / BEST_ROWS;
    const int n_it = (sp.Q + 31) >> 5;

    // The first loads of this warp's rows do not depend on the mask: they are issued before it is read.
    // Rows travel through a per-warp ring in shared memory filled by asynchronous 16-byte copies, so the
    // steps in flight cost no registers; a lane only ever reads the slots it filled itself.
    const float4 *row[BEST_ROWS];
    float4 *ring = reinterpret_cast<float4 *>(smem_raw) + (size_t(n_it) << 5) + size_t(warp) * (BEST_STAGES * BEST_ROWS * 32) + lane;
    auto set_rows = [&](int pr) {
        const int ca = pr * BEST_ROWS, n_rows = min(BEST_ROWS, sp.nC - ca);
#pragma unroll
        for (int k = 0; k < BEST_ROWS; ++k)
            row[k] = reinterpret_cast<const float4 *>(thr + (size_t(j) * sp.nC + ca + (k < n_rows ? k : 0)) * sp.P);
    };
    auto fetch = [&](int u, int it) {           // one group per step; lanes past the end re-read the last quad (their mask is 0)
        if (it < n_it) {
            const int q = min((it << 5) + lane, sp.Q - 1);
#pragma unroll
            for (int k = 0; k < BEST_ROWS; ++k)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::
                             "r"(uint32_t(__cvta_generic_to_shared(ring + (u * BEST_ROWS + k) * 32))), "l"(row[k] + q) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (warp < n_pairs) {
        set_rows(warp);
#pragma unroll
        for (int u = 0; u < BEST_STAGES; ++u) fetch(u, u);
    }

    for (int i = threadIdx.x; i < 2 * sp.nG; i += blockDim.x) { s_lo[i] = NO_LEVEL; s_hi[i] = -1; }
    for (int q = sp.Q + threadIdx.x; q < (n_it << 5); q += blockDim.x) maskf[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    bool bad = false, scattered = false;
    const uint4 *feas4 = reinterpret_cast<const uint4 *>(feas + size_t(j) * sp.P);
    for (int q0 = warp << 5; q0 < sp.Q; q0 += blockDim.x) {
        const int q = q0 + lane;
        int f[4] = {NO_LEVEL, NO_LEVEL, NO_LEVEL, NO_LEVEL};
        int g = 0;
        if (q < sp.Q) {
            const uint4 w4 = __ldg(feas4 + q);
            const uint32_t w[4] = {w4.x & full, w4.y & full, w4.z & full, w4.w & full};
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (w[k]) { f[k] = __ffs(w[k]) - 1; bad |= w[k] != ((full << f[k]) & full); }
            maskf[q] = make_float4(w[0] ? 1.f : 0.f, w[1] ? 1.f : 0.f, w[2] ? 1.f : 0.f, w[3] ? 1.f : 0.f);
            for (int k = 1; k < sp.nG; ++k) g += (4 * q >= sp.group_off[k]);
        }
        // one quad holds two plans of each class
        scattered |= (f[0] != NO_LEVEL && f[2] != NO_LEVEL && f[0] != f[2]) || (f[1] != NO_LEVEL && f[3] != NO_LEVEL && f[1] != f[3]);
        const int fe = min(f[0], f[2]), fo = min(f[1], f[3]);
        const int g0 = __shfl_sync(FULL, g, 0);
        if (__all_sync(FULL, g == g0 || q >= sp.Q)) {        // the usual case: the warp's quads lie in one GPU level
            const int lo_e = __reduce_min_sync(FULL, fe), lo_o = __reduce_min_sync(FULL, fo);
            const int hi_e = __reduce_max_sync(FULL, fe == NO_LEVEL ? -1 : fe), hi_o = __reduce_max_sync(FULL, fo == NO_LEVEL ? -1 : fo);
            if (lane == 0) {
                if (hi_e >= 0) { atomicMin(&s_lo[2 * g0], lo_e); atomicMax(&s_hi[2 * g0], hi_e); }
                if (hi_o >= 0) { atomicMin(&s_lo[2 * g0 + 1], lo_o); atomicMax(&s_hi[2 * g0 + 1], hi_o); }
            }
        } else if (q < sp.Q) {
            if (fe != NO_LEVEL) { atomicMin(&s_lo[2 * g], fe); atomicMax(&s_hi[2 * g], fe); }
            if (fo != NO_LEVEL) { atomicMin(&s_lo[2 * g + 1], fo); atomicMax(&s_hi[2 * g + 1], fo); }
        }
    }
    if (bad) atomicOr(status, DS_FEAS_NOT_THRESHOLD);
    __syncthreads();
    if (threadIdx.x < 2 * sp.nG) scattered |= s_hi[threadIdx.x] >= 0 && s_hi[threadIdx.x] != s_lo[threadIdx.x];
    if (__syncthreads_or(scattered)) {          // not the two-class shape: leave the job to the general kernel
        if (threadIdx.x == 0) todo[1 + atomicAdd(todo, 1)] = j;
        asm volatile("cp.async.wait_group 0;" ::: "memory");       // the copies issued above land before the CTA goes
        return;
    }

    const bool raw = (flags & RUBICK_BEST_RAW) != 0;
    const size_t o_step = size_t(sp.nC) * sp.nM;
    for (int pr = warp; pr < n_pairs; pr += n_warps) {
        const int ca = pr * BEST_ROWS;
        const int n_rows = min(BEST_ROWS, sp.nC - ca);          // the last group may be short
        if (pr != warp) {
            set_rows(pr);
#pragma unroll
            for (int u = 0; u < BEST_STAGES; ++u) fetch(u, u);
        }
        Best b;
        unsigned run_v[BEST_ROWS], run_i[BEST_ROWS];
        int run_g[BEST_ROWS];
#pragma unroll
        for (int k = 0; k < BEST_ROWS; ++k) {
            b.ev[k] = b.ov[k] = 0.f; b.ei[k] = b.oi[k] = -1;
            run_v[k] = 0u; run_i[k] = FULL; run_g[k] = 0;
        }
        int g = 0;                                  // GPU level being accumulated
        int g_end = sp.group_off[1] >> 2;           // its first quad past the end
        size_t o = (size_t(j) * sp.nG * sp.nC + ca) * sp.nM + lane;       // (j, g, ca, lane)

        // closes GPU level g for both rows: reductions, the two classes combined per memory level, curve, stores
        auto close_level = [&]() {
            const int fe = s_lo[2 * g], fo = s_lo[2 * g + 1];
            const int gv = sp.g_levels[g];
#pragma unroll
            for (int k = 0; k < BEST_ROWS; ++k) {
                const unsigned e_bits = __float_as_uint(b.ev[k]), o_bits = __float_as_uint(b.ov[k]);
                const unsigned me = __reduce_max_sync(FULL, e_bits), mo = __reduce_max_sync(FULL, o_bits);
                const unsigned ie = __reduce_min_sync(FULL, e_bits == me ? unsigned(b.ei[k]) : FULL);
                const unsigned io = __reduce_min_sync(FULL, o_bits == mo ? unsigned(b.oi[k]) : FULL);
                unsigned bv = lane >= fe ? me : 0u, bi = lane >= fe ? ie : FULL;
                const bool odd_wins = lane >= fo && (mo > bv || (mo == bv && io < bi));
                bv = odd_wins ? mo : bv; bi = odd_wins ? io : bi;
                int bg = bv ? gv : 0;               // the level's own plans use exactly its GPU count
                if (!raw) {
                    const bool up = bv > run_v[k];
                    run_v[k] = up ? bv : run_v[k]; run_i[k] = up ? bi : run_i[k]; run_g[k] = up ? bg : run_g[k];
                    bv = run_v[k]; bi = run_i[k]; bg = run_g[k];
                }
                if (k < n_rows && lane < sp.nM) {
                    const size_t ok = o + size_t(k) * sp.nM;
                    best_val[ok] = __uint_as_float(bv);
                    best_plan[ok] = int(bi);
                    best_g[ok] = bg;
                }
                b.ev[k] = b.ov[k] = 0.f; b.ei[k] = b.oi[k] = -1;
            }
            ++g;
            o += o_step;
            g_end = g < sp.nG ? sp.group_off[g + 1] >> 2 : 0x7fffffff;
        };

        for (int it0 = 0; it0 < n_it; it0 += BEST_STAGES) {
#pragma unroll
            for (int u = 0; u < BEST_STAGES; ++u) {
                const int it = it0 + u;
                if (it >= n_it) break;
                const int q = (it << 5) + lane;
                float4 v[BEST_ROWS];
                const float4 m = maskf[q];
                asm volatile("cp.async.wait_group %0;" :: "n"(BEST_STAGES - 1) : "memory");
#pragma unroll
                for (int k = 0; k < BEST_ROWS; ++k) v[k] = mul4(ring[(u * BEST_ROWS + k) * 32], m);
                fetch(u, it + BEST_STAGES);
                bool open = true;                   // this lane's quad has not been taken yet
                while (g_end <= (it << 5) + 32) {   // level g ends inside this step: its lanes first, then close it
                    accumulate(b, v, q, open && q < g_end);
                    open = q >= g_end;
                    close_level();
                }
                accumulate(b, v, q, open);
            }
        }
        while (g < sp.nG) close_level();            // levels without plans at the end of the list
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
}

typedef unsigned long long u64;

__device__ __forceinline__ u64 make_key(float v, int idx)
{
    return (static_cast<u64>(__float_as_uint(v)) << 32) | (0xffffffffu - uint32_t(idx));
}

struct Run {
    float v[BEST_ROWS]; int i[BEST_ROWS];
    uint32_t slot;            // 0xffff = nothing yet
};

__device__ __forceinline__ void run_flush(Run &r, u64 *bucket, int row_stride)
{
#pragma unroll
    for (int k = 0; k < BEST_ROWS; ++k) {
        if (r.v[k] > 0.0f) atomicMax(bucket + k * row_stride + r.slot, make_key(r.v[k], r.i[k]));
        r.v[k] = 0.0f; r.i[k] = -1;
    }
}

__device__ __forceinline__ void run_add(Run &r, u64 *bucket, int row_stride, uint32_t slot, int idx, const float (&val)[BEST_ROWS])
{
    if (slot == 0xffffu) return;
    if (slot != r.slot) { if (r.slot != 0xffffu) run_flush(r, bucket, row_stride); r.slot = slot; }
#pragma unroll
    for (int k = 0; k < BEST_ROWS; ++k)
        if (val[k] > r.v[k]) { r.v[k] = val[k]; r.i[k] = idx; }
}

__global__ void __launch_bounds__(BEST_WARPS * 32)
best_plan_scattered_kernel(const __grid_constant__ Space sp, const float *__restrict__ thr, const uint32_t *__restrict__ feas,
                           const int32_t *__restrict__ todo, unsigned flags, float *__restrict__ best_val,
                           int32_t *__restrict__ best_plan, int32_t *__restrict__ best_g, uint32_t *__restrict__ status)
{
  // todo[0] = number of jobs the streaming kernel left to this one, todo[1..] = their indices
  for (int li = blockIdx.x; li < todo[0]; li += gridDim.x) {
    __syncthreads();            // the previous job's shared memory is no longer read
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout: buckets [BEST_WARPS][BEST_ROWS][nG * 32] u64 | slot of every plan [P] u16
    const int row_stride = sp.nG * 32;
    const int n_warps = blockDim.x >> 5;
    u64 *buckets = reinterpret_cast<u64 *>(smem_raw);
    uint16_t *pslot = reinterpret_cast<uint16_t *>(buckets + size_t(n_warps) * BEST_ROWS * row_stride);

    const int j = todo[1 + li];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t full = sp.nM >= 32 ? 0xffffffffu : ((1u << sp.nM) - 1u);

    bool bad = false;
    for (int i = threadIdx.x; i < sp.P; i += blockDim.x) {
        const uint32_t w = __ldg(feas + size_t(j) * sp.P + i) & full;
        uint32_t s = 0xffffu;
        if (w) {
            const int f = __ffs(w) - 1;
            bad |= (w != ((full << f) & full));
            int g = 0;
            while (g + 1 < sp.nG && i >= sp.group_off[g + 1]) ++g;
            s = uint32_t(g * 32 + f);
        }
        pslot[i] = uint16_t(s);
    }
    if (bad) atomicOr(status, DS_FEAS_NOT_THRESHOLD);
    __syncthreads();

    u64 *bucket = buckets + size_t(warp) * BEST_ROWS * row_stride;
    const uint2 *pslot4 = reinterpret_cast<const uint2 *>(pslot);
    const bool raw = (flags & RUBICK_BEST_RAW) != 0;
    const int n_pairs = (sp.nC + BEST_ROWS - 1) / BEST_ROWS;

    for (int pr = warp; pr < n_pairs; pr += n_warps) {
        const int ca = pr * BEST_ROWS;
        const int n_rows = min(BEST_ROWS, sp.nC - ca);          // the last group may be short
        for (int i = lane; i < BEST_ROWS * row_stride; i += 32) bucket[i] = 0ull;
        __syncwarp();

        const float4 *row[BEST_ROWS];
#pragma unroll
        for (int k = 0; k < BEST_ROWS; ++k)
            row[k] = reinterpret_cast<const float4 *>(thr + (size_t(j) * sp.nC + ca + (k < n_rows ? k : 0)) * sp.P);
        Run even, odd;          // plans 4q, 4q+2 (no offload) / 4q+1, 4q+3 (offload)
        even.slot = odd.slot = 0xffffu;
#pragma unroll
        for (int k = 0; k < BEST_ROWS; ++k) { even.v[k] = odd.v[k] = 0.0f; even.i[k] = odd.i[k] = -1; }

        for (int q0 = lane; q0 < sp.Q; q0 += 32 * BEST_UNROLL) {
            float4 val[BEST_UNROLL][BEST_ROWS];
#pragma unroll
            for (int u = 0; u < BEST_UNROLL; ++u) {
                const int q = q0 + 32 * u;
#pragma unroll
                for (int k = 0; k < BEST_ROWS; ++k)
                    val[u][k] = q < sp.Q ? __ldcs(row[k] + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < BEST_UNROLL; ++u) {
                const int q = q0 + 32 * u;
                if (q >= sp.Q) break;
                const uint2 s4 = pslot4[q];
                float x[BEST_ROWS], y[BEST_ROWS], z[BEST_ROWS], w[BEST_ROWS];
#pragma unroll
                for (int k = 0; k < BEST_ROWS; ++k) { x[k] = val[u][k].x; y[k] = val[u][k].y; z[k] = val[u][k].z; w[k] = val[u][k].w; }
                run_add(even, bucket, row_stride, s4.x & 0xffffu, 4 * q + 0, x);
                run_add(odd, bucket, row_stride, s4.x >> 16, 4 * q + 1, y);
                run_add(even, bucket, row_stride, s4.y & 0xffffu, 4 * q + 2, z);
                run_add(odd, bucket, row_stride, s4.y >> 16, 4 * q + 3, w);
            }
        }
        if (even.slot != 0xffffu) run_flush(even, bucket, row_stride);
        if (odd.slot != 0xffffu) run_flush(odd, bucket, row_stride);
        __syncwarp();

#pragma unroll
        for (int k = 0; k < BEST_ROWS; ++k) {
            if (k >= n_rows) break;
            const int ci = ca + k;
            u64 running = 0ull;
            int running_g = 0;
            // outputs of (j, g, ci, lane) advance by nC * nM entries per GPU level
            size_t o = (size_t(j) * sp.nG * sp.nC + ci) * sp.nM + lane;
            const size_t o_step = size_t(sp.nC) * sp.nM;
            for (int g = 0; g < sp.nG; ++g, o += o_step) {
                const u64 mine = bucket[k * row_stride + g * 32 + lane];
                // best among plans whose first level is <= lane: maximum over the occupied buckets at or below
                unsigned occ = __ballot_sync(0xffffffffu, mine != 0ull);
                u64 best = 0ull;
                while (occ) {
                    const int f = __ffs(occ) - 1;
                    occ &= occ - 1;
                    const u64 ob = __shfl_sync(0xffffffffu, mine, f);
                    if (lane >= f && ob > best) best = ob;
                }
                int best_gv = best ? sp.g_levels[g] : 0;       // the level's own plans use exactly its GPU count
                if (!raw) {
                    if (best > running) { running = best; running_g = best_gv; }
                    best = running; best_gv = running_g;
                }
                if (lane < sp.nM) {
                    best_val[o] = best ? __uint_as_float(uint32_t(best >> 32)) : 0.0f;
                    best_plan[o] = best ? int(0xffffffffu - uint32_t(best)) : -1;
                    best_g[o] = best_gv;
                }
            }
        }
        __syncwarp();
    }
  }
}

// every job goes to the general kernel (plan lists whose masks do not fit the streaming kernel's shared memory)
__global__ void best_plan_todo_all_kernel(int32_t *__restrict__ todo, int J)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) todo[0] = J;
    if (i < J) todo[1 + i] = i;
}

static int best_warps(const Space &sp)
{
    const int pairs = (sp.nC + BEST_ROWS - 1) / BEST_ROWS;
    return pairs < BEST_WARPS ? pairs : BEST_WARPS;
}

static int scattered_warps(const Space &sp)
{
    const size_t budget = 200 * 1024, plan_bytes = (size_t(sp.P) * 2 + 15) & ~size_t(15);
    const size_t per_warp = size_t(BEST_ROWS) * sp.nG * 32 * 8;
    int w = plan_bytes < budget ? int((budget - plan_bytes) / per_warp) : 0;
    const int pairs = (sp.nC + BEST_ROWS - 1) / BEST_ROWS;
    if (w > BEST_WARPS) w = BEST_WARPS;
    if (w > pairs) w = pairs;
    return w;
}

// d_todo: J + 1 words of scratch (count, then the jobs left to the general kernel)
cudaError_t launch_best(const Space &sp, const float *d_thr, const uint32_t *d_feas, int J, unsigned flags,
                        float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g, uint32_t *d_status,
                        int32_t *d_todo, int num_sms, cudaStream_t st)
{
    if (J == 0) return cudaSuccess;
    const int warps = best_warps(sp), warps2 = scattered_warps(sp);
    if (warps2 < 1) return cudaErrorInvalidConfiguration;     // plan list too long for one CTA's shared memory
    const size_t smem = (size_t((sp.Q + 31) & ~31) + size_t(warps) * BEST_STAGES * BEST_ROWS * 32) * sizeof(float4);
    const size_t smem2 = size_t(warps2) * BEST_ROWS * sp.nG * 32 * 8 + ((size_t(sp.P) * 2 + 15) & ~size_t(15));
    cudaError_t e;
    if (smem > 48 * 1024 && smem <= 200 * 1024) {
        e = cudaFuncSetAttribute(best_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
    }
    if (smem2 > 48 * 1024) {
        e = cudaFuncSetAttribute(best_plan_scattered_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem2));
        if (e != cudaSuccess) return e;
    }
    if (smem <= 200 * 1024) {
        e = cudaMemsetAsync(d_todo, 0, sizeof(int32_t), st);
        if (e != cudaSuccess) return e;
        best_plan_kernel<<<J, warps * 32, smem, st>>>(sp, d_thr, d_feas, J, flags, d_best_val, d_best_plan, d_best_g, d_status, d_todo); count_launch();
    } else {
        best_plan_todo_all_kernel<<<(J + 255) / 256, 256, 0, st>>>(d_todo, J); count_launch();
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int grid2 = J < 2 * num_sms ? J : 2 * num_sms;
    best_plan_scattered_kernel<<<grid2, warps2 * 32, smem2, st>>>(sp, d_thr, d_feas, d_todo, flags, d_best_val, d_best_plan, d_best_g, d_status); count_launch();
    return cudaGetLastError();
}

}  // namespace rubick
