// Candidate-grid evaluation: predicted throughput for every (job, plan, CPU level) and the
// memory-feasibility word for every (job, plan).
//
// Mapping.  Plans come in quads: four consecutive plan indices share (d, t, p, ZeRO stage) and
// differ in (gradient checkpointing, offload) = (0,0), (0,1), (1,0), (1,1).  One thread owns one
// (job, quad): it reads the 128-byte job record once, computes everything that does not depend
// on the CPU level once (forward / backward time, the three communication times, T_cc, the
// non-offload optimizer time, the offload transfer time and its overlap with the gradient
// ring), then walks the CPU levels and stores one float4 per level.  Consecutive threads own
// consecutive quads, so a warp writes 512 contiguous bytes per level: the kernel is a pure
// write stream of 4 bytes per candidate plus 4 / C bytes of mask.  Four consecutive quads are the
// ZeRO stages 0..3 of one (d, t, p) triple; their lanes split the per-level transcendental work.
//
// Model (paper Section 4):  THROUGHPUT = b / T_iter,  T_iter = T_cc + T_oo + k_const  (Eq. 1)
//   T_fwd  = tau * mu / (t p) * (m + p - 1 if p > 1)                       forward, pipeline bubble
//   T_bwd  = k_bwd T_fwd (+ T_fwd under gradient checkpointing)
//   T_comm = V / B per dimension, V = 0 at degree 1;  V_dp ring all-reduce of the shard (every ZeRO stage),
//            V_tp four all-reduces per layer, V_pp stage boundaries of 1F1B
//   T_cc   = a T_fwd + (a - 1) T_bwd + f^{k_sync}(T_bwd, T_dp) + T_tp + T_pp
//   T_oo   = T_opt, or under ZeRO-Offload f^{k_off}(T_dp, T_off) + f^{k_swap}(T_opt(c), T_off)
//   f^k(x, y) = (x^k + y^k)^(1/k)                                           (Section 4.3)
// Arithmetic is single precision.  f^k is evaluated as M (1 + (m/M)^k)^(1/k) with M = max and
// m = min, so that no power can overflow and the hardware log2 / exp2 approximations act on
// arguments where their absolute error stays below 1e-6 relative to the result.
//
// Feasibility (integer bytes, exact): mixed-precision Adam model states (2 + 2 + 12 bytes per
// shard parameter, ZeRO stage 1 / 2 / 3 dividing optimizer / + gradients / + parameters by d,
// offload moving gradients and optimizer states to the host), activations of one stage's layers
// for the micro-batches in flight, against the GPU memory; host need g * host_base (+ 14 P under
// offload) against each host-memory level and its per-node share against the node.

#include "rubick_internal.cuh"

namespace rubick {

__device__ __forceinline__ float lg2_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^-n for 0 <= n < 127, exact
__device__ __forceinline__ float pow2_neg(int n) { return __int_as_float((127 - n) << 23); }

// f^k(x, y) for x, y >= 0 with inv_k = 1 / k
__device__ __forceinline__ float overlap(float k, float inv_k, float x, float y)
{
    float hi = fmaxf(x, y), lo = fminf(x, y);
    if (lo == 0.0f) return hi;
    float r = lo * rcp_approx(hi);               // in (0, 1]
    float u = ex2_approx(k * lg2_approx(r));     // r^k in [0, 1]
    return hi * ex2_approx(inv_k * lg2_approx(1.0f + u));
}

__device__ __forceinline__ int64_t cdiv_shift(int64_t x, int s) { return (x + ((int64_t(1) << s) - 1)) >> s; }

struct JobRegs {
    double P; int64_t host_base;
    int32_t l, h, s, b, mu_cap, alpha;
    float tau, k_bwd, k_sync, k_opt, k_opt_off, k_off, k_swap, k_const;
};

__device__ __forceinline__ JobRegs load_job(const rubick_job *jp)
{
    const int4 *v = reinterpret_cast<const int4 *>(jp);
    int4 a = __ldg(v + 0), b = __ldg(v + 1), c = __ldg(v + 2), d = __ldg(v + 3), e = __ldg(v + 4);
    JobRegs r;
    r.P = __hiloint2double(a.y, a.x);
    r.host_base = (int64_t(uint32_t(a.w)) << 32) | uint32_t(a.z);
    r.l = b.x; r.h = b.y; r.s = b.z; r.b = b.w;
    r.mu_cap = c.x; r.alpha = c.y; r.tau = __int_as_float(c.z); r.k_bwd = __int_as_float(c.w);
    r.k_sync = __int_as_float(d.x); r.k_opt = __int_as_float(d.y); r.k_opt_off = __int_as_float(d.z);
    r.k_off = __int_as_float(d.w);
    r.k_swap = __int_as_float(e.x); r.k_const = __int_as_float(e.y);
    return r;
}

// first level index whose value is >= need (nM if none); levels strictly increasing
__device__ __forceinline__ int first_level(const Space &sp, int64_t need)
{
    int lo = 0, hi = sp.nM;
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (sp.m_levels[mid] >= need) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// What the offload plans of a quad (stage >= 2: plans 4q + 1 and 4q + 3) need per core level c:
//   throughput = bf * rcp(base_i + f^{k_swap}(opt_c / c, T_off)),  i = 0 without / 1 with gradient checkpointing
struct OffloadTerms {
    float T_off, opt_c;        // transfer time; optimizer time on one core (the same on the four quads of a triple)
    float base0, base1;        // everything else in T_iter, per checkpointing setting
    float k_swap, inv_kswap, bf;
    bool ok0, ok1;             // plan 4q + 1 / 4q + 3 is structurally valid and not disabled
    bool any;                  // some lane of the warp holds such a plan (warp-uniform)
};

// Everything one thread does for (job j, quad q): the feasibility words (stored by active threads) and the
// four throughputs of every CPU level, handed to emit(ci, float4, words) in ascending level order.  Whole warps
// must call this together with the quads of a warp consecutive and starting at a multiple of four (the
// four ZeRO stages of a (d, t, p) triple trade results); `active` = false for mirror threads past the end.
// Returns the four feasibility words when KEEP_WORDS (zeros otherwise).
// WIDE: degrees of any size from the wide quad table (divisions); otherwise powers of two from the
// logarithms of the quad table (shifts, exact reciprocals).
// TERMS_ONLY: the caller walks the core levels itself: head(out, words, terms) is called once with the two
// throughputs that do not depend on the core count (out.x, out.z), the quad's four words and the quad's terms of the
// offload plans (OffloadTerms; the same bits the float4 form uses), and emit is never called.
template <bool KEEP_WORDS, bool WIDE, bool TERMS_ONLY, class Head, class Emit>
__device__ __forceinline__ uint4 eval_quad(const Space &sp, const void *__restrict__ quads_any,
                                           const rubick_job *__restrict__ jobs, int j, int q, bool active,
                                           uint32_t *__restrict__ feas, Head &&head, Emit &&emit)
{
    const JobRegs jb = load_job(jobs + j);
    int ld = 0, lt = 0, lp = 0, lg = 0, accum = 0, d, t, p, z, qflags, disabled;
    if constexpr (WIDE) {
        const uint4 qraw = __ldg(reinterpret_cast<const uint4 *>(quads_any) + q);
        d = qraw.x & 0xffff; t = qraw.x >> 16; p = qraw.y & 0xffff; z = (qraw.y >> 16) & 0xff; accum = qraw.y >> 24;
        qflags = qraw.z & 0xff; disabled = (qraw.z >> 8) & 0xff;
    } else {
        const uint2 qraw = __ldg(reinterpret_cast<const uint2 *>(quads_any) + q);
        ld = qraw.x & 0xff; lt = (qraw.x >> 8) & 0xff; lp = (qraw.x >> 16) & 0xff; z = (qraw.x >> 24) & 0xff;
        qflags = (qraw.y >> 8) & 0xff; disabled = (qraw.y >> 16) & 0xff;
        lg = ld + lt + lp;
        d = 1 << ld; t = 1 << lt; p = 1 << lp;
    }
    const int g = d * t * p;
    // x / divisor rounded up; the divisor is 1 << shift in the power-of-two space
    auto cdiv_by = [](int64_t x, int divisor, int shift) -> int64_t {
        if constexpr (WIDE) return (x + divisor - 1) / divisor; else return cdiv_shift(x, shift);
    };

    // structural validity of the (d, t, p, z) part; offload additionally needs ZeRO stage >= 2
    bool valid = (qflags & QF_T_FITS_NODE) && p <= jb.l && d <= jb.b && !(sp.strict && z > 0 && (t > 1 || p > 1));
    if constexpr (WIDE) valid = valid && jb.b % d == 0 && jb.h % t == 0;
    else valid = valid && (jb.b & (d - 1)) == 0 && (jb.h & (t - 1)) == 0;
    // micro-batching
    const int r = max(WIDE ? jb.b / d : jb.b >> ld, 1);
    // explicit accumulation (wide space): the micro-batch halved `accum` times; it must still hold a sample
    const int mu_most = min(r, max(jb.mu_cap, 1));
    const int mu = max(mu_most >> accum, 1);
    if constexpr (WIDE) valid = valid && (mu_most >> accum) >= 1;
    const bool valid_off = valid && z >= 2;
    const int n = (r + mu - 1) / mu;
    const int m = p > 1 ? n : 1;
    const int a = p > 1 ? 1 : n;

    // ---- times that do not depend on the CPU level -------------------------------------------
    const float inv_tp = WIDE ? 1.0f / float(t * p) : pow2_neg(lt + lp);
    const float inv_dt = WIDE ? 1.0f / float(d * t) : pow2_neg(ld + lt);
    float T_fwd = jb.tau * float(mu) * inv_tp;
    if (p > 1) T_fwd *= float(n + p - 1);
    const float T_bwd0 = jb.k_bwd * T_fwd;
    const float T_bwd1 = T_bwd0 + T_fwd;

    const float Pf = float(jb.P);
    const float bsh = float(int64_t(jb.b) * jb.s * jb.h);
    float T_dp = 0.0f, T_tp = 0.0f, T_pp = 0.0f;
    if (d > 1) {
        float V = sp.e * Pf * (WIDE ? 2.0f * float(d - 1) / float(g) : float(d - 1) * pow2_neg(lg - 1));
        if (z == 3) V *= sp.z3_volume;                   // 1 unless the environment asks for stage 3's parameter gathers
        T_dp = V * ((qflags & QF_DP_INTER) ? sp.inv_B_inter : sp.inv_B_intra);
    }
    if (t > 1) T_tp = sp.e * 8.0f * float(t - 1) * bsh * float(jb.l) * inv_dt * sp.inv_B_intra;
    if (p > 1) T_pp = sp.e * 2.0f * float(p) * bsh * inv_dt * ((qflags & QF_PP_INTER) ? sp.inv_B_inter : sp.inv_B_intra);

    const float inv_ksync = 1.0f / jb.k_sync;
    const float af = float(a);
    const float fixed = af * T_fwd + T_tp + T_pp + jb.k_const;
    const float cc0 = fixed + (af - 1.0f) * T_bwd0 + overlap(jb.k_sync, inv_ksync, T_bwd0, T_dp);
    const float cc1 = fixed + (af - 1.0f) * T_bwd1 + overlap(jb.k_sync, inv_ksync, T_bwd1, T_dp);

    const float Psi = Pf * inv_tp;
    const float inv_d = WIDE ? 1.0f / float(d) : pow2_neg(ld);
    const float T_opt = jb.k_opt * Psi * (z >= 1 ? inv_d : 1.0f);
    const float bf = float(jb.b);

    uint4 fw_out = make_uint4(0u, 0u, 0u, 0u);
    float4 out;
    out.x = (valid && !(disabled & 1)) ? bf / (cc0 + T_opt) : 0.0f;
    out.z = (valid && !(disabled & 4)) ? bf / (cc1 + T_opt) : 0.0f;
    out.y = 0.0f;
    out.w = 0.0f;

    // ---- feasibility words ---------------------------------------------------------------------
    {
        const int64_t Pi = int64_t(jb.P);
        const int64_t Psi_i = cdiv_by(Pi, t * p, lt + lp);
        const int64_t Psi_d = cdiv_by(Psi_i, d, ld);              // the shard of a ZeRO-partitioned state
        const int64_t params = 2 * (z == 3 ? Psi_d : Psi_i);
        const int64_t grads = 2 * (z >= 2 ? Psi_d : Psi_i);
        const int64_t opt = 12 * (z >= 1 ? Psi_d : Psi_i);
        const int64_t smh = int64_t(jb.s) * mu * jb.h;
        const int64_t A = cdiv_by(int64_t(jb.alpha) * smh, t, lt);
        const int64_t Lq = cdiv_by(jb.l, p, lp) * (p > 1 ? min(m, p) : 1);
        const int64_t act0 = Lq * A;
        const int64_t act1 = Lq * 2 * smh + A;
        const int64_t st0 = params + grads + opt, st1 = params;
        const int64_t need0 = WIDE ? jb.host_base * g : jb.host_base << lg;
        const int64_t need1 = need0 + 14 * Pi;
        const int nshift = max(lg - sp.log2Gn, 0);
        const int nodes = g > sp.Gn ? g / sp.Gn : 1;
        const uint32_t full = sp.nM >= 32 ? 0xffffffffu : ((1u << sp.nM) - 1u);
        uint32_t w0 = 0u, w1 = 0u;
        if (cdiv_by(need0, nodes, nshift) <= sp.Mn) { int f = first_level(sp, need0); if (f < sp.nM) w0 = (full << f) & full; }
        if (cdiv_by(need1, nodes, nshift) <= sp.Mn) { int f = first_level(sp, need1); if (f < sp.nM) w1 = (full << f) & full; }
        uint4 fw;
        fw.x = (valid && !(disabled & 1) && st0 + act0 <= sp.gpu_mem) ? w0 : 0u;
        fw.y = (valid_off && !(disabled & 2) && st1 + act0 <= sp.gpu_mem) ? w1 : 0u;
        fw.z = (valid && !(disabled & 4) && st0 + act1 <= sp.gpu_mem) ? w0 : 0u;
        fw.w = (valid_off && !(disabled & 8) && st1 + act1 <= sp.gpu_mem) ? w1 : 0u;
        if (active) *reinterpret_cast<uint4 *>(feas + (size_t(j) * sp.P + 4 * size_t(q))) = fw;
        if (KEEP_WORDS) fw_out = fw;
    }

    // ---- walk the CPU levels -------------------------------------------------------------------
    // The four lanes of a triple (ZeRO stages 0..3 of the same d, t, p) share the work that depends on
    // the core count: the swap overlap f^{k_swap}(T_opt(c), T_off) is the same for all four offload
    // plans of the triple, so lane i evaluates it for core level 4n + i and the lanes trade results;
    // then every lane divides for ONE offload plan (stage 2 + (lane >> 1), checkpointing = lane & 1)
    // and the two lanes that own offload plans (stages 2 and 3) collect their pair.
    const bool off0 = valid_off && !(disabled & 2), off1 = valid_off && !(disabled & 8);
    const unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31, gbase = lane & ~3, zl = lane & 3;
    const bool any_off = __any_sync(FULL, off0 || off1);
    if (!any_off) {
        if constexpr (TERMS_ONLY) head(out, fw_out, OffloadTerms{0.0f, 0.0f, 0.0f, 0.0f, 1.0f, 1.0f, bf, false, false, false});
        else for (int ci = 0; ci < sp.nC; ++ci) emit(ci, out, fw_out);
        return fw_out;
    }
    const float T_off = sp.e * Psi * inv_d * sp.inv_B_pcie;          // identical on the four lanes
    const float opt_c = jb.k_opt_off * Psi * inv_d;                  // times 1 / c
    const float inv_kswap = 1.0f / jb.k_swap;
    float base0 = 0.0f, base1 = 0.0f;
    if (valid_off) {
        const float f_off = overlap(jb.k_off, 1.0f / jb.k_off, T_dp, T_off);
        base0 = cc0 + f_off; base1 = cc1 + f_off;
    }
    if constexpr (TERMS_ONLY) {
        head(out, fw_out, OffloadTerms{T_off, opt_c, base0, base1, jb.k_swap, inv_kswap, bf, off0, off1, true});
        return fw_out;
    }
    const int src = gbase + 2 + (zl >> 1);
    const float sb0 = __shfl_sync(FULL, base0, src), sb1 = __shfl_sync(FULL, base1, src);
    const int okbits = __shfl_sync(FULL, (off0 ? 1 : 0) | (off1 ? 2 : 0), src);
    const float my_base = (zl & 1) ? sb1 : sb0;
    const bool my_ok = (okbits >> (zl & 1)) & 1;
    const int src_y = gbase + (zl == 3 ? 2 : 0), src_w = gbase + (zl == 3 ? 3 : 1);
    for (int c0 = 0; c0 < sp.nC; c0 += 4) {
        const int ci_mine = min(c0 + zl, sp.nC - 1);
        const float fs_mine = overlap(jb.k_swap, inv_kswap, opt_c * sp.inv_c[ci_mine], T_off);
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
            const float fs = __shfl_sync(FULL, fs_mine, gbase + cc);
            const float r = my_ok ? bf * rcp_approx(my_base + fs) : 0.0f;
            const float ry = __shfl_sync(FULL, r, src_y), rw = __shfl_sync(FULL, r, src_w);
            if (c0 + cc < sp.nC) {
                out.y = zl >= 2 ? ry : 0.0f;
                out.w = zl >= 2 ? rw : 0.0f;
                emit(c0 + cc, out, fw_out);
            }
        }
    }
    return fw_out;
}

template <bool WIDE>
__global__ void __launch_bounds__(256)
eval_candidates_kernel(const __grid_constant__ Space sp, const void *__restrict__ quads,
                       const rubick_job *__restrict__ jobs, int J, float *__restrict__ thr,
                       uint32_t *__restrict__ feas)
{
    // J * Q < 2^31 is checked by the host entry point
    // Threads past the end mirror the last valid thread and store nothing: the CPU-level walk
    // exchanges values between the four lanes of a (d, t, p) triple, so whole warps stay converged.
    const uint32_t total = uint32_t(J) * uint32_t(sp.Q);
    const uint32_t gid_raw = blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = gid_raw < total;
    const uint32_t gid = active ? gid_raw : total - 1;
    const int j = int(gid / uint32_t(sp.Q));
    const int q = int(gid - uint32_t(j) * uint32_t(sp.Q));
    float *row = thr + (size_t(j) * sp.nC * sp.P + 4 * size_t(q));
    // levels arrive in ascending order, one call each: the row pointer just advances
    eval_quad<false, WIDE, false>(sp, quads, jobs, j, q, active, feas, [](const float4 &, const uint4 &, const OffloadTerms &) {},
                                  [&](int, const float4 &out, const uint4 &) {
        if (active) __stcs(reinterpret_cast<float4 *>(row), out);
        row += sp.P;
    });
}

// ------------------------------------------------------------------------------------------------------
// Curves without the table: the evaluation above and the best-plan / sensitivity-curve step (paper
// Section 5.2) in one kernel, for callers that only want the curves (a scheduling round).  One CTA per
// job, and nothing but the mask (4 bytes per plan) and the curves goes to memory.
//
// Pass over 32 quads per warp, in two parts.  (1) Lane = quad, as in the table kernel: the feasibility words and
// everything that does not depend on the core count.  Plans without offload do not depend on it at all: per
// GPU level their maximum is one warp reduction over the quads' two values and a vote that names the lowest lane
// holding it (quads ascend with the lane, so that is the lowest plan index).  (2) Lane = core level: the eight
// (d, t, p) triples of the pass are walked one after the other, their terms handed round by shuffles; every
// lane evaluates the triple's four offload plans at its own core level, in plan order, and keeps the running
// maximum and its plan index in registers (strictly greater replaces: lowest index on ties).  No reduction
// across lanes is needed, and the values are the same bits as the table kernel's.  Where the GPU level
// changes inside a pass, and at its end, lane c folds its (value bits << 32 | ~index) into the slot
// (GPU level, core level c) of its warp with a plain read-compare-write: a slot of the offload class only ever
// has that one writer.
//
// After a CTA barrier the warps' slots are merged; then the output phase combines the two classes per memory
// level (under this library's memory rule the plans of a class share one first feasible memory level per GPU
// level), takes the running maximum over GPU levels and stores value, plan and GPU count: four memory levels per
// thread with 16-byte stores when the layout allows it.  Same values, same ties (lowest plan index) as best_plan
// on the table of eval_candidates: bit-identical.
// ------------------------------------------------------------------------------------------------------
constexpr int CURVES_THREADS = 128;      // small CTAs: the phases of the several CTAs of an SM overlap
constexpr int CURVES_WARPS = CURVES_THREADS / 32;
constexpr int CURVES_MIN_CTAS = 10;      // registers capped at 48 a thread: 40 warps an SM hide the shuffle and reciprocal latencies (0.57 ms against 0.89 ms uncapped)

template <bool WIDE, bool VEC4>
__global__ void __launch_bounds__(CURVES_THREADS, WIDE ? 8 : CURVES_MIN_CTAS)       // the wide instance needs 64 registers
curves_kernel(const __grid_constant__ Space sp, const QuadDesc *__restrict__ quads, const void *__restrict__ quads_any,
              const rubick_job *__restrict__ jobs, int J, unsigned flags, uint32_t *__restrict__ feas,
              float *__restrict__ best_val, int32_t *__restrict__ best_plan, int32_t *__restrict__ best_g, int4 *__restrict__ top)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // [warp][nG][nC + 1]: offload class per core level, then the other class; warp 0's copy receives the merge
    unsigned long long *keys = reinterpret_cast<unsigned long long *>(smem_raw);
    __shared__ int s_first[2 * RUBICK_MAX_G_LEVELS];        // first feasible memory level per (GPU level, class), nM = none
    __shared__ float s_inv_c[RUBICK_MAX_C_LEVELS];          // lane-indexed look-ups: not from the constant bank
    const int j = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned FULL = 0xffffffffu;
    const int per_warp = sp.nG * (sp.nC + 1);

    for (int i = tid; i < CURVES_WARPS * per_warp; i += blockDim.x) keys[i] = 0ull;
    if (tid < sp.nC) s_inv_c[tid] = sp.inv_c[tid];
    if (tid < sp.nG) {
        // host-memory need of the level's plans: g processes, plus the offloaded states (as in the mask above)
        const rubick_job *jp = jobs + j;
        const int g = sp.g_levels[tid];
        const int64_t need0 = jp->host_base_bytes * g, need1 = need0 + 14 * int64_t(jp->P);
        const int nodes = g > sp.Gn ? g / sp.Gn : 1;
        int f0 = sp.nM, f1 = sp.nM;
        if ((need0 + nodes - 1) / nodes <= sp.Mn) f0 = first_level(sp, need0);
        if ((need1 + nodes - 1) / nodes <= sp.Mn) f1 = first_level(sp, need1);
        s_first[2 * tid] = f0; s_first[2 * tid + 1] = f1;
    }
    __syncthreads();

    unsigned long long *mine = keys + size_t(warp) * per_warp;
    for (int q0 = 0; q0 < sp.Q; q0 += blockDim.x) {
        const int q_raw = q0 + tid;
        const bool active = q_raw < sp.Q;
        if (q0 + (tid & ~31) >= sp.Q) continue;                 // a whole warp past the end has nothing to mirror
        const int q = active ? q_raw : sp.Q - 1;
        const int level = reinterpret_cast<const uint8_t *>(quads + q)[4];             // QuadDesc::g_level
        const unsigned peers = __match_any_sync(FULL, active ? level : -1);            // lanes of the same GPU level
        const int q_lane0 = q_raw - lane;                       // quad of lane 0 (quads ascend with the lane)
        OffloadTerms ot;
        unsigned has1 = 0u, has3 = 0u;                          // lanes whose plan 4q + 1 / 4q + 3 may run at some memory level
        eval_quad<true, WIDE, true>(sp, quads_any, jobs, j, q, active, feas,
            [&](const float4 &o, const uint4 &words, const OffloadTerms &terms) {
                // plans without offload: the quad's two values; infeasible plans count as 0
                ot = terms;
                const float x = words.x ? o.x : 0.0f, z = words.z ? o.z : 0.0f;
                const unsigned be = active ? __float_as_uint(fmaxf(x, z)) : 0u;
                const unsigned me = __reduce_max_sync(peers, be);
                const unsigned who = __ballot_sync(peers, be == me) & peers;
                const unsigned second = __ballot_sync(peers, z > x);
                if (me && lane == __ffs(peers) - 1) {
                    const int wl = __ffs(who) - 1;
                    const unsigned idx = 4u * unsigned(q_lane0 + wl) + (((second >> wl) & 1u) ? 2u : 0u);
                    const unsigned long long key = (static_cast<unsigned long long>(me) << 32) | (FULL - idx);
                    unsigned long long *slot = mine + size_t(level) * (sp.nC + 1) + sp.nC;
                    if (key > *slot) *slot = key;
                }
                has1 = __ballot_sync(FULL, active && terms.ok0 && words.y != 0u);
                has3 = __ballot_sync(FULL, active && terms.ok1 && words.w != 0u);
            },
            [](int, const float4 &, const uint4 &) {});
        if (ot.any && ((has1 | has3) != 0u)) {
            // lane = core level: walk the pass's triples (lanes 4 tau .. 4 tau + 3 hold ZeRO stages 0..3; the offload
            // plans are those of stages 2 and 3)
            for (int cb = 0; cb < sp.nC; cb += 32) {
                const int ci = cb + lane;
                const bool have = ci < sp.nC;
                const float inv_c = s_inv_c[have ? ci : 0];
                float run_v = 0.0f; unsigned run_i = 0u;
                int cur = __shfl_sync(FULL, level, 0);
                auto flush = [&](int lvl) {
                    if (have && run_v > 0.0f) {
                        const unsigned long long key = (static_cast<unsigned long long>(__float_as_uint(run_v)) << 32) | (FULL - run_i);
                        unsigned long long *slot = mine + size_t(lvl) * (sp.nC + 1) + ci;
                        if (key > *slot) *slot = key;
                    }
                    run_v = 0.0f;
                };
#pragma unroll 2
                for (int tau = 0; tau < 8; ++tau) {
                    const int l0 = 4 * tau;
                    const unsigned bits = (((has1 >> (l0 + 2)) & 1u)) | (((has3 >> (l0 + 2)) & 1u) << 1)
                                        | (((has1 >> (l0 + 3)) & 1u) << 2) | (((has3 >> (l0 + 3)) & 1u) << 3);     // warp-uniform
                    const int lvl = __shfl_sync(FULL, level, l0);
                    if (lvl != cur) { flush(cur); cur = lvl; }
                    if (!bits) continue;
                    const float T_off = __shfl_sync(FULL, ot.T_off, l0 + 2), opt_c = __shfl_sync(FULL, ot.opt_c, l0 + 2);
                    const float b20 = __shfl_sync(FULL, ot.base0, l0 + 2), b21 = __shfl_sync(FULL, ot.base1, l0 + 2);
                    const float b30 = __shfl_sync(FULL, ot.base0, l0 + 3), b31 = __shfl_sync(FULL, ot.base1, l0 + 3);
                    const float fs = overlap(ot.k_swap, ot.inv_kswap, opt_c * inv_c, T_off);
                    const unsigned p2 = 4u * unsigned(q_lane0 + l0 + 2), p3 = p2 + 4u;
                    // the four plans in index order; strictly greater replaces
                    if (bits & 1u) { const float r = ot.bf * rcp_approx(b20 + fs); if (r > run_v) { run_v = r; run_i = p2 + 1u; } }
                    if (bits & 2u) { const float r = ot.bf * rcp_approx(b21 + fs); if (r > run_v) { run_v = r; run_i = p2 + 3u; } }
                    if (bits & 4u) { const float r = ot.bf * rcp_approx(b30 + fs); if (r > run_v) { run_v = r; run_i = p3 + 1u; } }
                    if (bits & 8u) { const float r = ot.bf * rcp_approx(b31 + fs); if (r > run_v) { run_v = r; run_i = p3 + 3u; } }
                }
                flush(cur);
            }
        }
        __syncwarp();                                           // the slot of the other class may have another writer in the next pass
    }
    __syncthreads();
    // merge the warps' slots into warp 0's
    for (int i = tid; i < per_warp; i += blockDim.x) {
        unsigned long long k = keys[i];
#pragma unroll
        for (int w = 1; w < CURVES_WARPS; ++w) { const unsigned long long o = keys[size_t(w) * per_warp + i]; k = o > k ? o : k; }
        keys[i] = k;
    }
    __syncthreads();

    const bool raw = (flags & RUBICK_BEST_RAW) != 0;
    // what (GPU level g, core level ci) offers at memory level m: the better of the two classes that may run there
    auto entry = [&](int g, unsigned long long ke, unsigned long long ko, int fe, int fo, int m, unsigned &bv, unsigned &bi, int &bg) {
        const bool use_e = ke && m >= fe, use_o = ko && m >= fo;
        bv = use_e ? unsigned(ke >> 32) : 0u; bi = use_e ? FULL - unsigned(ke) : FULL;
        const unsigned vo = unsigned(ko >> 32), io = FULL - unsigned(ko);
        const bool odd_wins = use_o && (vo > bv || (vo == bv && io < bi));
        bv = odd_wins ? vo : bv; bi = odd_wins ? io : bi;
        bg = bv ? sp.g_levels[g] : 0;
    };
    if constexpr (VEC4) {
        // nM is a multiple of 4 and the three tables are 16-byte aligned: one thread = four memory levels
        const int m4 = sp.nM >> 2;
        for (int item = tid; item < sp.nC * m4; item += blockDim.x) {
            const int ci = item / m4, mb = (item - ci * m4) << 2;
            unsigned run_v[4] = {0u, 0u, 0u, 0u}, run_i[4] = {FULL, FULL, FULL, FULL}; int run_g[4] = {0, 0, 0, 0};
            size_t o = (size_t(j) * sp.nG * sp.nC + ci) * sp.nM + mb;
            for (int g = 0; g < sp.nG; ++g, o += size_t(sp.nC) * sp.nM) {
                const unsigned long long ke = keys[size_t(g) * (sp.nC + 1) + sp.nC], ko = keys[size_t(g) * (sp.nC + 1) + ci];
                const int fe = s_first[2 * g], fo = s_first[2 * g + 1];
                uint4 v; int4 pi, gg;
                unsigned *vv = reinterpret_cast<unsigned *>(&v); int *pp = reinterpret_cast<int *>(&pi), *gp = reinterpret_cast<int *>(&gg);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    unsigned bv, bi; int bg;
                    entry(g, ke, ko, fe, fo, mb + k, bv, bi, bg);
                    if (!raw) {
                        const bool up = bv > run_v[k];
                        run_v[k] = up ? bv : run_v[k]; run_i[k] = up ? bi : run_i[k]; run_g[k] = up ? bg : run_g[k];
                        bv = run_v[k]; bi = run_i[k]; bg = run_g[k];
                    }
                    vv[k] = bv; pp[k] = int(bi); gp[k] = bg;
                }
                *reinterpret_cast<uint4 *>(best_val + o) = v;
                *reinterpret_cast<int4 *>(best_plan + o) = pi;
                *reinterpret_cast<int4 *>(best_g + o) = gg;
                // the top memory level once more, packed, when the caller asked for it
                if (top && mb + 4 == sp.nM) top[(size_t(j) * sp.nG + g) * sp.nC + ci] = make_int4(int(vv[3]), pp[3], gp[3], 0);
            }
        }
    } else {
        for (int cm = tid; cm < sp.nC * sp.nM; cm += blockDim.x) {
            const int ci = cm / sp.nM, m = cm - ci * sp.nM;
            unsigned run_v = 0u, run_i = FULL; int run_g = 0;
            size_t o = (size_t(j) * sp.nG * sp.nC + ci) * sp.nM + m;
            for (int g = 0; g < sp.nG; ++g, o += size_t(sp.nC) * sp.nM) {
                const unsigned long long ke = keys[size_t(g) * (sp.nC + 1) + sp.nC], ko = keys[size_t(g) * (sp.nC + 1) + ci];
                unsigned bv, bi; int bg;
                entry(g, ke, ko, s_first[2 * g], s_first[2 * g + 1], m, bv, bi, bg);
                if (!raw) {
                    const bool up = bv > run_v;
                    run_v = up ? bv : run_v; run_i = up ? bi : run_i; run_g = up ? bg : run_g;
                    bv = run_v; bi = run_i; bg = run_g;
                }
                best_val[o] = __uint_as_float(bv);
                best_plan[o] = int(bi);
                best_g[o] = bg;
                if (top && m == sp.nM - 1) top[(size_t(j) * sp.nG + g) * sp.nC + ci] = make_int4(int(bv), int(bi), bg, 0);
            }
        }
    }
}

cudaError_t launch_curves(const Space &sp, const QuadDesc *d_quads, const void *d_wide_quads, const rubick_job *d_jobs, int J,
                          unsigned flags, uint32_t *d_feas, float *d_best_val, int32_t *d_best_plan, int32_t *d_best_g,
                          cudaStream_t st, int4 *d_top)
{
    if (J == 0) return cudaSuccess;
    const size_t smem = size_t(CURVES_WARPS) * sp.nG * (sp.nC + 1) * sizeof(unsigned long long);
    // 16-byte stores of four memory levels need rows that start on 16-byte boundaries
    const bool vec4 = (sp.nM & 3) == 0 && ((reinterpret_cast<uintptr_t>(d_best_val) | reinterpret_cast<uintptr_t>(d_best_plan)
                                            | reinterpret_cast<uintptr_t>(d_best_g)) & 15) == 0;
    auto launch = [&](auto kernel, const void *quads_any) -> cudaError_t {
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
            if (e != cudaSuccess) return e;
        }
        kernel<<<J, CURVES_THREADS, smem, st>>>(sp, d_quads, quads_any, d_jobs, J, flags, d_feas, d_best_val, d_best_plan, d_best_g, d_top);
        count_launch();
        return cudaGetLastError();
    };
    if (sp.wide) return vec4 ? launch(curves_kernel<true, true>, d_wide_quads) : launch(curves_kernel<true, false>, d_wide_quads);
    return vec4 ? launch(curves_kernel<false, true>, d_quads) : launch(curves_kernel<false, false>, d_quads);
}

cudaError_t launch_eval(const Space &sp, const QuadDesc *d_quads, const void *d_wide_quads, const rubick_job *d_jobs, int J,
                        float *d_thr, uint32_t *d_feas, cudaStream_t st)
{
    if (J == 0) return cudaSuccess;
    const int64_t total = int64_t(J) * sp.Q;
    const int block = 256;
    const int64_t grid = (total + block - 1) / block;
    if (sp.wide) eval_candidates_kernel<true><<<unsigned(grid), block, 0, st>>>(sp, d_wide_quads, d_jobs, J, d_thr, d_feas);
    else eval_candidates_kernel<false><<<unsigned(grid), block, 0, st>>>(sp, d_quads, d_jobs, J, d_thr, d_feas);
    count_launch();
    return cudaGetLastError();
}

}  // namespace rubick
