// Best plan per (job, GPU level, CPU level, host-memory level) and the resource-sensitivity
// curve (paper Section 5.2): an argmax over the plans of one GPU level that are feasible at a
// memory level, lowest plan index on ties, then the running maximum along the GPU axis.
//
// One CTA owns one job.  Its feasibility words are turned once into "first feasible level" bytes
// in shared memory (words are thresholds in the level index, so the first set bit says it all).
// Each warp then takes CPU levels in turn: lanes stream the level's row of the throughput table
// with 16-byte loads (four plans = one quad per load) and keep, per lane, a running maximum for
// the (GPU level, first feasible level) pair they are currently seeing; when the pair changes the
// run is pushed into a per-warp bucket array [GPU level][memory level] with a 64-bit shared-memory
// max.  Candidates are ordered by the 64-bit key (value bits << 32 | ~plan index): positive floats
// order like their bit patterns, and the inverted index makes the lowest plan win equal values.
// After the row, lane m owns memory level m: a shuffle prefix-maximum over lanes turns buckets
// into "best among plans feasible at level <= m", and a running maximum over GPU levels gives the
// curve.  The table is read once (4 bytes per candidate); outputs are 12 bytes per (g, c, m).

#include "rubick_internal.cuh"

namespace rubick {

constexpr int BEST_WARPS = 8;

__device__ __forceinline__ unsigned long long make_key(float v, int idx)
{
    return (static_cast<unsigned long long>(__float_as_uint(v)) << 32) | (0xffffffffu - uint32_t(idx));
}

struct Run {
    unsigned long long key;   // 0 = empty
    int slot;                 // g_level * 32 + first level
};

__device__ __forceinline__ void run_flush(Run &r, unsigned long long *bucket)
{
    if (r.key) atomicMax(bucket + r.slot, r.key);
    r.key = 0ull;
}

__device__ __forceinline__ void run_add(Run &r, unsigned long long *bucket, float v, int idx, int f, int grp)
{
    if (f == 255 || !(v > 0.0f)) return;
    const int slot = grp * 32 + f;
    const unsigned long long k = make_key(v, idx);
    if (slot != r.slot) { run_flush(r, bucket); r.slot = slot; }
    r.key = k > r.key ? k : r.key;
}

__global__ void __launch_bounds__(BEST_WARPS * 32)
best_plan_kernel(const __grid_constant__ Space sp, const float *__restrict__ thr, const uint32_t *__restrict__ feas,
                 int J, unsigned flags, float *__restrict__ best_val, int32_t *__restrict__ best_plan,
                 int32_t *__restrict__ best_g, uint32_t *__restrict__ status)
{
    extern __shared__ unsigned char smem_raw[];
    // layout: buckets [BEST_WARPS][nG][32] u64 | first level [P] u8 (padded to 4) | quad group [Q] u8
    unsigned long long *buckets = reinterpret_cast<unsigned long long *>(smem_raw);
    uint8_t *flevel = reinterpret_cast<uint8_t *>(buckets + BEST_WARPS * sp.nG * 32);
    uint8_t *qgroup = flevel + ((sp.P + 15) & ~15);

    const int j = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t full = sp.nM >= 32 ? 0xffffffffu : ((1u << sp.nM) - 1u);

    bool bad = false;
    for (int i = threadIdx.x; i < sp.P; i += blockDim.x) {
        const uint32_t w = __ldg(feas + size_t(j) * sp.P + i) & full;
        int f = 255;
        if (w) {
            f = __ffs(w) - 1;
            bad |= (w != ((full << f) & full));
        }
        flevel[i] = uint8_t(f);
    }
    for (int q = threadIdx.x; q < sp.Q; q += blockDim.x) {
        int g = 0;
        while (g + 1 < sp.nG && 4 * q >= sp.group_off[g + 1]) ++g;
        qgroup[q] = uint8_t(g);
    }
    if (bad) atomicOr(status, DS_FEAS_NOT_THRESHOLD);
    __syncthreads();

    unsigned long long *bucket = buckets + warp * sp.nG * 32;
    const uint32_t *flevel4 = reinterpret_cast<const uint32_t *>(flevel);
    const bool raw = (flags & RUBICK_BEST_RAW) != 0;

    for (int ci = warp; ci < sp.nC; ci += BEST_WARPS) {
        for (int i = lane; i < sp.nG * 32; i += 32) bucket[i] = 0ull;
        __syncwarp();

        const float4 *row = reinterpret_cast<const float4 *>(thr + (size_t(j) * sp.nC + ci) * sp.P);
        Run even = {0ull, -1}, odd = {0ull, -1};   // plans 4q, 4q+2 (no offload) / 4q+1, 4q+3 (offload)
        constexpr int UNROLL = 4;
        for (int q0 = lane; q0 < sp.Q; q0 += 32 * UNROLL) {
            float4 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int q = q0 + 32 * u;
                v[u] = q < sp.Q ? __ldcs(row + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int q = q0 + 32 * u;
                if (q >= sp.Q) break;
                const uint32_t f4 = flevel4[q];
                const int grp = qgroup[q];
                run_add(even, bucket, v[u].x, 4 * q + 0, f4 & 0xff, grp);
                run_add(odd, bucket, v[u].y, 4 * q + 1, (f4 >> 8) & 0xff, grp);
                run_add(even, bucket, v[u].z, 4 * q + 2, (f4 >> 16) & 0xff, grp);
                run_add(odd, bucket, v[u].w, 4 * q + 3, f4 >> 24, grp);
            }
        }
        run_flush(even, bucket);
        run_flush(odd, bucket);
        __syncwarp();

        unsigned long long running = 0ull;
        for (int g = 0; g < sp.nG; ++g) {
            unsigned long long k = bucket[g * 32 + lane];
            // inclusive prefix maximum over lanes: best among plans whose first level is <= lane
#pragma unroll
            for (int s = 1; s < 32; s <<= 1) {
                const unsigned long long o = __shfl_up_sync(0xffffffffu, k, s);
                if (lane >= s && o > k) k = o;
            }
            if (!raw) { running = k > running ? k : running; k = running; }
            if (lane < sp.nM) {
                const size_t o = ((size_t(j) * sp.nG + g) * sp.nC + ci) * sp.nM + lane;
                const int plan = k ? int(0xffffffffu - uint32_t(k)) : -1;
                best_val[o] = k ? __uint_as_float(uint32_t(k >> 32)) : 0.0f;
                best_plan[o] = plan;
                best_g[o] = plan >= 0 ? sp.g_levels[qgroup[plan >> 2]] : 0;
            }
        }
        __syncwarp();
    }
}

size_t best_smem_bytes(const Space &sp)
{
    return size_t(BEST_WARPS) * sp.nG * 32 * 8 + ((sp.P + 15) & ~15) + ((sp.Q + 15) & ~15);
}

cudaError_t launch_best(const Space &sp, const float *d_thr, const uint32_t *d_feas, int J, unsigned flags,
                        float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g, uint32_t *d_status,
                        cudaStream_t st)
{
    if (J == 0) return cudaSuccess;
    const size_t smem = best_smem_bytes(sp);
    static size_t configured = 0;
    if (smem > 48 * 1024 && smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(best_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        configured = smem;
    }
    best_plan_kernel<<<J, BEST_WARPS * 32, smem, st>>>(sp, d_thr, d_feas, J, flags, d_best_val, d_best_plan,
                                                       d_best_g, d_status);
    return cudaGetLastError();
}

}  // namespace rubick
