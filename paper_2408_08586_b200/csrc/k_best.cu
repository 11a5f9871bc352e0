// Best plan per (job, GPU level, CPU level, host-memory level) and the resource-sensitivity
// curve (paper Section 5.2): an argmax over the plans of one GPU level that are feasible at a
// memory level, lowest plan index on ties, then the running maximum along the GPU axis.
//
// One CTA owns one job.  Its feasibility words are turned once into 16-bit "slots" in shared memory:
// slot = GPU level * 32 + first feasible memory level (words are thresholds in the level index, so
// the first set bit says it all), 0xffff for a plan that is feasible nowhere.  Each warp then takes
// BEST_ROWS CPU levels at a time: lanes stream both rows of the throughput table with 16-byte loads (four
// plans = one quad per load) and keep, per row and per plan parity (offload plans alternate with
// the others and usually need another memory level), a running (value, index) maximum for the slot
// they are currently seeing; a strict "greater" keeps the lowest index because a lane meets its
// plans in ascending order.  When the slot changes, the run is pushed into a per-warp bucket array
// [row][slot] with a 64-bit shared-memory max on (value bits << 32 | ~index): positive floats order
// like their bit patterns and the inverted index makes the lowest plan win equal values across
// lanes.  After the rows, lane m owns memory level m: the maximum over the occupied buckets at or
// below m gives "best among plans feasible at level m", and a running maximum over GPU levels
// gives the curve.  The table is read once (4 bytes per candidate); outputs are 12 bytes per
// (g, c, m).

#include "rubick_internal.cuh"

namespace rubick {

constexpr int BEST_WARPS = 12;         // at most; fewer when the buckets of many GPU levels would not fit
constexpr int BEST_ROWS = 2;          // CPU levels a warp processes together
constexpr int BEST_UNROLL = 2;        // quads per lane in flight per row

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
best_plan_kernel(const __grid_constant__ Space sp, const float *__restrict__ thr, const uint32_t *__restrict__ feas,
                 int J, unsigned flags, float *__restrict__ best_val, int32_t *__restrict__ best_plan,
                 int32_t *__restrict__ best_g, uint32_t *__restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout: buckets [BEST_WARPS][BEST_ROWS][nG * 32] u64 | slot of every plan [P] u16
    const int row_stride = sp.nG * 32;
    const int n_warps = blockDim.x >> 5;
    u64 *buckets = reinterpret_cast<u64 *>(smem_raw);
    uint16_t *pslot = reinterpret_cast<uint16_t *>(buckets + size_t(n_warps) * BEST_ROWS * row_stride);

    const int j = blockIdx.x;
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

static int best_warps(const Space &sp)
{
    const size_t budget = 200 * 1024, plan_bytes = (size_t(sp.P) * 2 + 15) & ~size_t(15);
    const size_t per_warp = size_t(BEST_ROWS) * sp.nG * 32 * 8;
    int w = plan_bytes < budget ? int((budget - plan_bytes) / per_warp) : 0;
    const int pairs = (sp.nC + BEST_ROWS - 1) / BEST_ROWS;
    if (w > BEST_WARPS) w = BEST_WARPS;
    if (w > pairs) w = pairs;
    return w;
}

cudaError_t launch_best(const Space &sp, const float *d_thr, const uint32_t *d_feas, int J, unsigned flags,
                        float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g, uint32_t *d_status,
                        cudaStream_t st)
{
    if (J == 0) return cudaSuccess;
    const int warps = best_warps(sp);
    if (warps < 1) return cudaErrorInvalidConfiguration;      // plan list too long for one CTA's shared memory
    const size_t smem = size_t(warps) * BEST_ROWS * sp.nG * 32 * 8 + ((size_t(sp.P) * 2 + 15) & ~size_t(15));
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(best_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
    }
    best_plan_kernel<<<J, warps * 32, smem, st>>>(sp, d_thr, d_feas, J, flags, d_best_val, d_best_plan, d_best_g, d_status);
    return cudaGetLastError();
}

}  // namespace rubick
