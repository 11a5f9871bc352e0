// Machine probes: four micro-kernels that measure, on the GPU the library runs on, the rates its kernels are
// compared with -- a write-only stream, a read-only stream, single-precision fused multiply-adds and the
// transcendental unit (lg2 / ex2 / rcp approximations).  The benchmark times them with CUDA events and quotes
// roofline fractions against them; nothing on the scheduling path calls them.

#include "rubick_internal.cuh"

namespace rubick {

std::atomic<unsigned long long> g_kernel_launches{0};

// float4 streaming stores over the whole buffer, grid-stride
__global__ void __launch_bounds__(256) probe_write_kernel(float4 *__restrict__ buf, size_t n4)
{
    const float4 v = make_float4(1.0f, 2.0f, 3.0f, 4.0f);
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < n4; i += size_t(gridDim.x) * blockDim.x)
        __stcs(buf + i, v);
}

// float4 streaming loads over the whole buffer; one word per thread keeps the loads alive
__global__ void __launch_bounds__(256) probe_read_kernel(const float4 *__restrict__ buf, size_t n4, float *__restrict__ sink)
{
    float acc = 0.0f;
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < n4; i += size_t(gridDim.x) * blockDim.x) {
        const float4 v = __ldcs(buf + i);
        acc += (v.x + v.y) + (v.z + v.w);
    }
    if (acc == 123.456f) sink[0] = acc;            // never true for the probe's contents; defeats dead-code removal
}

constexpr int PROBE_CHAINS = 8;                    // independent dependency chains per thread

// PROBE_CHAINS independent chains of fused multiply-adds per thread, `iters` rounds of 4 per chain
__global__ void __launch_bounds__(256) probe_fma_kernel(int iters, float *__restrict__ sink)
{
    float x[PROBE_CHAINS];
#pragma unroll
    for (int c = 0; c < PROBE_CHAINS; ++c) x[c] = 1.0f + 1e-3f * float(threadIdx.x + c);
    const float a = 0.999f, b = 1e-3f;
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < PROBE_CHAINS; ++c) x[c] = fmaf(x[c], a, b);
    }
    float s = 0.0f;
#pragma unroll
    for (int c = 0; c < PROBE_CHAINS; ++c) s += x[c];
    if (s == 123.456f) sink[0] = s;
}

// PROBE_CHAINS independent chains of lg2 -> ex2 -> rcp per thread (the three approximations the evaluation uses)
__global__ void __launch_bounds__(256) probe_xu_kernel(int iters, float *__restrict__ sink)
{
    float x[PROBE_CHAINS];
#pragma unroll
    for (int c = 0; c < PROBE_CHAINS; ++c) x[c] = 1.5f + 1e-3f * float(threadIdx.x + c);
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int c = 0; c < PROBE_CHAINS; ++c) {
            float y;
            asm volatile("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x[c]));
            asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(y));
            asm volatile("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(y));
            x[c] = y;
        }
    }
    float s = 0.0f;
#pragma unroll
    for (int c = 0; c < PROBE_CHAINS; ++c) s += x[c];
    if (s == 123.456f) sink[0] = s;
}

}  // namespace rubick

using namespace rubick;

extern "C" int rubick_probe(rubick_ctx *ctx, int kind, void *d_buf, size_t bytes, int iters, double *h_work)
{
    if (!ctx) return RUBICK_EINVAL;
    if (!d_buf || bytes < 4096 || (reinterpret_cast<uintptr_t>(d_buf) & 15)) return fail(ctx, RUBICK_EINVAL, "probe: a 16-byte aligned buffer of at least 4096 bytes");
    if (iters < 1 || iters > (1 << 24)) return fail(ctx, RUBICK_EINVAL, "probe: 1 .. 2^24 iterations");
    if (cudaSetDevice(ctx->device) != cudaSuccess) return fail(ctx, RUBICK_ECUDA, "cudaSetDevice failed");
    const int threads = 256;
    const int grid = ctx->num_sms * 8;               // eight resident CTAs of 256 threads per SM
    const size_t n4 = bytes / 16;
    double work = 0.0;
    switch (kind) {
    case RUBICK_PROBE_WRITE:
        probe_write_kernel<<<grid, threads, 0, ctx->stream>>>(static_cast<float4 *>(d_buf), n4);
        work = double(n4) * 16.0;
        break;
    case RUBICK_PROBE_READ:
        probe_read_kernel<<<grid, threads, 0, ctx->stream>>>(static_cast<const float4 *>(d_buf), n4, static_cast<float *>(d_buf));
        work = double(n4) * 16.0;
        break;
    case RUBICK_PROBE_FMA:
        probe_fma_kernel<<<grid, threads, 0, ctx->stream>>>(iters, static_cast<float *>(d_buf));
        work = double(grid) * threads * double(iters) * 4.0 * PROBE_CHAINS;
        break;
    case RUBICK_PROBE_XU:
        probe_xu_kernel<<<grid, threads, 0, ctx->stream>>>(iters, static_cast<float *>(d_buf));
        work = double(grid) * threads * double(iters) * 3.0 * PROBE_CHAINS;
        break;
    default:
        return fail(ctx, RUBICK_EINVAL, "probe: unknown kind");
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch probe");
    g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    if (h_work) *h_work = work;
    return RUBICK_OK;
}

extern "C" unsigned long long rubick_kernel_launches(void)
{
    return g_kernel_launches.load(std::memory_order_relaxed);
}
