// CenteredClip streaming passes (App. D.2, eq. (CenteredClip)) for sm_100a.
//
// One pass reads the [P][n][row_stride] tensor exactly once.  A CTA owns a contiguous range of
// column tiles of one partition; a thread keeps R rows x 4 columns of the current tile in
// registers (R independent 128-bit loads in flight), so that the update of v and the residual
// norms at the *updated* v come out of the same registers:
//
//   weights w_i from the norms the previous pass left behind      (prologue, per CTA)
//   u[c]  = (1/n) sum_i w_i (x_i[c] - v[c]);  v'[c] = v[c] + u[c]  (eq. (CenteredClip))
//   norm2_i += (x_i[c] - v'[c])^2;  step2 += u[c]^2               (feeds the next pass)
//
// Cross-CTA sums are not floating-point atomics: every CTA writes its partial sums to its own slot,
// and the CTA of a partition that finishes last (an integer ticket, nobody waits) adds the slots in
// a fixed order, so results are reproducible run to run.  The stop rule is evaluated the same way
// by every CTA of a partition at the top of the next pass, from those totals.
#include <type_traits>

#include "btard_common.h"
#include "btard_median.cuh"

namespace btard {
namespace {

// 128-bit read-only load with an L2 eviction policy (from createpolicy).
__device__ __forceinline__ float4 ld_policy(const float* p, uint64_t policy)
{
    float4 r;
    asm volatile("ld.global.nc.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p), "l"(policy));
    return r;
}
__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ uint64_t policy_evict_last()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ double warp_sum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    return x;
}

// Clip weight min{1, tau/rho} from the squared norm; non-finite norms give 0.
__device__ __forceinline__ float clip_weight(double norm2, double tau, bool& nonfinite)
{
    const double rho = sqrt(norm2);
    if (!isfinite(rho)) { nonfinite = true; return 0.0f; }
    if (rho <= tau) return 1.0f;
    return (float)(tau / rho);
}

// Weights of the rows for the next update, from their squared residual norms (all threads call it;
// it ends with the CTA synchronised).  CenteredClip: min{1, tau / rho}.  Geometric median (Weiszfeld):
// n (1/rho_i) / sum_j (1/rho_j), rho floored at tau, so that (1/n) sum_i w_i (x_i - v) is the
// Weiszfeld step.  Rows with a non-finite norm get 0 and raise *sh_flag.  scratch: n doubles.
__device__ void row_weights(const double* sh_sum, float* sh_w, int n, double tau, int rule, int* sh_flag,
                            double* scratch)
{
    const int tid = threadIdx.x;
    if (rule == BTARD_RULE_GEOMETRIC_MEDIAN) {
        for (int i = tid; i < n; i += blockDim.x) {
            const double rho = sqrt(sh_sum[i]);
            double inv = 0.0;
            if (isfinite(rho)) inv = 1.0 / fmax(rho, tau);
            else *sh_flag = 1;
            scratch[i] = inv;
        }
        __syncthreads();
        double total = 0.0;
        for (int i = 0; i < n; ++i) total += scratch[i];           // same order in every thread
        for (int i = tid; i < BTARD_MAX_PEERS + 16; i += blockDim.x)
            sh_w[i] = (i < n && total > 0.0) ? (float)((double)n * scratch[i] / total) : 0.0f;
    } else {
        for (int i = tid; i < BTARD_MAX_PEERS + 16; i += blockDim.x) {
            bool bad = false;
            sh_w[i] = (i < n) ? clip_weight(sh_sum[i], tau, bad) : 0.0f;
            if (bad) *sh_flag = 1;
        }
    }
    __syncthreads();
}

struct KernelArgs {
    CclipLaunch a;
    int RG, CL, cpp;
};

// Records the end state of a partition (called by one CTA of it).
__device__ void finish_partition(const CclipLaunch& a, int p, const double* sums, int iters_done,
                                 bool eps_mode)
{
    const int n = a.n;
    for (int i = threadIdx.x; i < n; i += blockDim.x) a.resid_norm[(size_t)p * n + i] = sqrt(sums[i]);
    if (threadIdx.x == 0) {
        const double step2 = sums[n];
        a.iters[p] = iters_done;
        a.last_step[p] = sqrt(step2);
        unsigned st = 0;
        for (int i = 0; i < n; ++i)
            if (!isfinite(sums[i])) st |= BTARD_STATUS_NONFINITE_ROW;
        if (eps_mode && !(step2 <= a.eps2)) st |= BTARD_STATUS_NOT_CONVERGED;
        atomicOr(&a.status[p], st);
        a.done[p] = 1;
    }
}

// bf16 <-> fp32 for the low-order part of v (round to nearest even; inputs are finite and tiny).
__device__ __forceinline__ uint32_t bf16_bits(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ float bf16_value(uint32_t b) { return __uint_as_float(b << 16); }

// v + s as an unevaluated sum hi + lo (Knuth's TwoSum), lo then rounded to bf16.
__device__ __forceinline__ void two_sum_bf16(float v, float s, float& hi, float& lo, uint32_t& lo_bits)
{
    hi = __fadd_rn(v, s);
    const float bb = __fadd_rn(hi, -v);
    const float err = __fadd_rn(__fadd_rn(v, -__fadd_rn(hi, -bb)), __fadd_rn(s, -bb));
    lo_bits = bf16_bits(err);
    lo = bf16_value(lo_bits);
}

// Two fp32 values in one 64-bit register, and the packed arithmetic on them.
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// 128-bit load of a row as two packed pairs: read-only, streaming (evicted first).  The streaming
// qualifier instead of a policy operand saves the per-load move of the policy into a uniform register
// (measured: 2-3 % per update at n = 16 and n = 64 with rows that fit L2 partly, nothing at d = 2^28).
__device__ __forceinline__ void ld_row_pairs(const float* p, uint64_t& lo, uint64_t& hi)
{
    asm volatile("ld.global.cs.nc.v2.b64 {%0, %1}, [%2];" : "=l"(lo), "=l"(hi) : "l"(p));
}

// COMP (PASS_ITER only): v is carried as hi + lo, hi the fp32 output vector and lo a bf16 correction
// in the workspace, so that the update and the stop test do not drown in the rounding of v.
template <int R, int MODE, bool COMP>
__global__ void __launch_bounds__(512) cclip_pass_kernel(const KernelArgs k)
{
    extern __shared__ float4 sh_x[];                  // [2][RG][CL] exchange of partial column sums
    __shared__ double sh_sum[BTARD_MAX_PEERS + 1];
    __shared__ float sh_w[BTARD_MAX_PEERS + 16];      // zero beyond row n - 1
    __shared__ double sh_red[16][17];
    __shared__ double sh_part[512 + BTARD_MAX_PEERS + 1];
    __shared__ int sh_flag;
    __shared__ float sh_wsum;                         // sum of the clip weights (PASS_ITER)
    __shared__ __align__(8) float2 sh_w2[(MODE == PASS_ITER) ? BTARD_MAX_PEERS + 16 : 1];   // (w_i, w_i)
    __shared__ float sh_f[BTARD_MAX_PEERS + 16];      // row factors (with row_scale)

    const CclipLaunch& a = k.a;
    const int n = a.n, RG = k.RG, CL = k.CL, cpp = k.cpp;
    const bool scaled = a.row_scale != nullptr;       // rows enter as f_i x_i: the guarded tile path applies f
    const int tid = threadIdx.x, cl = tid % CL, rg = tid / CL;
    // Consecutive passes sweep the tensor in opposite directions, so that a pass starts on the
    // lines the previous one touched last and finds part of them still in L2.
    constexpr bool UPDATE = (MODE == PASS_ITER || MODE == PASS_COMBINE);   // v moves in this pass
    const bool rev = (MODE == PASS_ITER) && ((a.l & 1) == 0);
    const int bid = rev ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x;
    const int p = bid / cpp, j = bid % cpp;
    const long long stride = a.stride;
    const long long len = a.table[p].len;
    const double tau = a.table[p].tau;

    const float* gp = a.g + (size_t)p * n * stride;
    const float* xrow0 = gp + (size_t)(rg * R) * stride;   // this thread's first row; one stride per further row
    const long long stride_bytes = stride * 4;
    const int nrows = (n - rg * R < R) ? n - rg * R : R;   // rows of this group that exist
    float* vp = a.v + (size_t)p * stride;
    unsigned short* lop = COMP ? a.v_lo + (size_t)p * stride : nullptr;
    const float inv_n = 1.0f / (float)n;

    // This CTA's share of the partition, in groups of 4 columns ("quads"), cut on 128-byte lines.
    const long long Q = stride >> 2;
    long long q0 = Q * j / cpp, q1 = Q * (j + 1) / cpp;
    if (j > 0) q0 &= ~7LL;
    if (j + 1 < cpp) q1 &= ~7LL;
    const long long full_quads = len >> 2;             // quads that lie entirely inside the data
    const long long ntiles = (q1 - q0 + CL - 1) / CL;
    // The rows are marked evict-first in L2: nothing is read twice within a pass, and what is
    // still resident when the next pass starts (it starts where this one ends) is a bonus.
    // Measured: pinning the tail with evict-last instead was slower for every budget tried.
    const uint64_t pol = policy_evict_first();

    // Update passes are launched back to back with programmatic dependent launch: this grid may start
    // while the previous pass is still draining.  Until griddepcontrol.wait returns, only memory that
    // no pass writes is touched: the partition table and the rows of g.  The rows of the first tile
    // are asked into L2 here, so that they are on their way while the previous pass finishes and
    // while the clip weights are worked out below.  (done[p] only ever goes from 0 to 1 between the
    // start pass and here, so a 1 read early is final and a 0 is checked again after the wait.)
    if (MODE == PASS_ITER) {
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        if (ntiles > 0 && tid < n && !*reinterpret_cast<const volatile int*>(a.done + p)) {
            const long long qb = q0 + (rev ? ntiles - 1 : 0) * CL;
            const long long rest = q1 - qb;
            const unsigned bytes = (unsigned)(rest < CL ? rest : CL) * 16u;
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(gp + (size_t)tid * stride + qb * 4), "r"(bytes) : "memory");
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    if (scaled) {                                     // row_scale is an input: nothing in the chain of passes writes it
        for (int i = threadIdx.x; i < BTARD_MAX_PEERS + 16; i += blockDim.x)
            sh_f[i] = (i < n) ? (float)a.row_scale[(size_t)p * n + i] : 0.0f;
    }
    if (MODE == PASS_ITER) {
        if (a.done[p]) return;
        // Totals the previous pass left behind: squared norms at the current v, and its squared step.
        const double* src = a.tot_in + (size_t)p * (n + 1);
        for (int i = tid; i <= n; i += blockDim.x) sh_sum[i] = __ldcg(src + i);
        __syncthreads();
        const bool converged = (a.stop_mode == BTARD_STOP_EPS) && a.l >= 1 && (sh_sum[n] <= a.eps2);
        if (converged) {                              // same decision in every CTA of the partition
            if (j == 0) finish_partition(k.a, p, sh_sum, a.l, true);
            return;
        }
        if (tid == 0) sh_flag = 0;
        __syncthreads();
        // the radius of this update: the schedule's tau_l when one is given
        const double tau_l = a.tau_sched ? a.tau_sched[(size_t)p * a.max_iters + a.l] : tau;
        row_weights(sh_sum, sh_w, n, tau_l, a.rule, &sh_flag, sh_part);
        if (tid == 0) {
            float w = 0.0f;
            for (int i = 0; i < n; ++i) w += sh_w[i];
            sh_wsum = w;
            if (j == 0 && sh_flag) atomicOr(&a.status[p], BTARD_STATUS_NONFINITE_ROW);
        }
        __syncthreads();
    } else if (MODE == PASS_COMBINE) {
        // v = v0 + sum_i a_i (x_i - v0): the update formula with weights n a_i.
        for (int i = tid; i < BTARD_MAX_PEERS + 16; i += blockDim.x)
            sh_w[i] = (i < n) ? (float)((double)n * a.coef[(size_t)p * n + i]) : 0.0f;
        __syncthreads();
    } else if (MODE == PASS_INIT) {
        if (j == 0 && tid == 0) { a.done[p] = 0; a.status[p] = 0; }
    }
    (void)tau;
    const float* wrow = sh_w + rg * R;                // this thread's R clip weights
    bool skip_rows = false;                           // some row has weight 0 and must be left out
    if (MODE == PASS_ITER) {
        for (int i = tid; i < BTARD_MAX_PEERS + 16; i += blockDim.x) sh_w2[i] = make_float2(sh_w[i], sh_w[i]);
        skip_rows = sh_flag != 0;
        __syncthreads();
    }

    if (scaled) __syncthreads();                      // the row factors are in shared memory

    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.0f;
    float step_acc = 0.0f;

    // v is read and written by every update pass: its loads ask L2 to keep the lines and its stores are
    // marked streaming (measured: fewer DRAM bytes and a shorter pass than with default accesses).
    // Only while v (all partitions) fits well inside L2; a larger v streams like the rows.
    constexpr bool KEEPV = (MODE == PASS_ITER);
    const uint64_t keep = a.v_fits_l2 ? policy_evict_last() : policy_evict_first();
    // One tile: CL quads starting at quad qb.  MASKED = false when every lane's quad is inside both
    // the CTA's range and the data, so no predicate is needed.
    auto tile = [&](auto masked_tag, long long qb, int parity, uint64_t policy) {
        constexpr bool MASKED = decltype(masked_tag)::value;
        const long long col = (qb + cl) * 4;
        const bool valid = !MASKED || (qb + cl < q1);
        const bool m0 = !MASKED || (valid && col < len), m1 = !MASKED || (valid && col + 1 < len);
        const bool m2 = !MASKED || (valid && col + 2 < len), m3 = !MASKED || (valid && col + 3 < len);
        float4 x[R];
        float4 v4 = make_float4(0.f, 0.f, 0.f, 0.f);
        float4 lo4 = make_float4(0.f, 0.f, 0.f, 0.f);      // low-order part of v (COMP)
        if (valid) {
            const char* xr = reinterpret_cast<const char*>(xrow0 + col);
#pragma unroll
            for (int r = 0; r < R; ++r, xr += stride_bytes)
                x[r] = (r < nrows) ? ld_policy(reinterpret_cast<const float*>(xr), policy) : make_float4(0.f, 0.f, 0.f, 0.f);
            if (scaled) {
#pragma unroll
                for (int r = 0; r < R; ++r) x[r] = scale_row(x[r], sh_f[rg * R + r]);
            }
            if (MODE != PASS_INIT || a.init_mode == BTARD_INIT_CALLER_V0) {
                if (KEEPV) asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;" : "=f"(v4.x), "=f"(v4.y), "=f"(v4.z), "=f"(v4.w) : "l"(vp + col), "l"(keep));
                else v4 = *reinterpret_cast<const float4*>(vp + col);
            }
            if (COMP) {
                uint2 lb;
                if (KEEPV) asm volatile("ld.global.L2::cache_hint.v2.u32 {%0, %1}, [%2], %3;" : "=r"(lb.x), "=r"(lb.y) : "l"(lop + col), "l"(keep));
                else lb = *reinterpret_cast<const uint2*>(lop + col);
                lo4 = make_float4(bf16_value(lb.x & 0xFFFFu), bf16_value(lb.x >> 16),
                                  bf16_value(lb.y & 0xFFFFu), bf16_value(lb.y >> 16));
            }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) x[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (MODE != PASS_INIT) {                       // residuals at the current v
#pragma unroll
            for (int r = 0; r < R; ++r) {
                x[r].x = (x[r].x - v4.x) - lo4.x; x[r].y = (x[r].y - v4.y) - lo4.y;
                x[r].z = (x[r].z - v4.z) - lo4.z; x[r].w = (x[r].w - v4.w) - lo4.w;
            }
        }

        float4 vn = v4;                                // v after this pass
        float4 dv = make_float4(0.f, 0.f, 0.f, 0.f);   // what the represented v moved by
        if (UPDATE || (MODE == PASS_INIT && a.init_mode == BTARD_INIT_MEAN)) {
            float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (UPDATE) {
                    const float wr = wrow[r];
                    if (wr != 0.0f) {                  // weight 0: the row is left out, not multiplied
                        s4.x = fmaf(wr, x[r].x, s4.x); s4.y = fmaf(wr, x[r].y, s4.y);
                        s4.z = fmaf(wr, x[r].z, s4.z); s4.w = fmaf(wr, x[r].w, s4.w);
                    }
                } else {
                    s4.x += x[r].x; s4.y += x[r].y; s4.z += x[r].z; s4.w += x[r].w;
                }
            }
            if (RG > 1) {                              // add the row groups' partial column sums
                float4* buf = sh_x + (size_t)parity * RG * CL;
                buf[rg * CL + cl] = s4;
                __syncthreads();
                s4 = buf[cl];
                for (int q = 1; q < RG; ++q) {
                    const float4 o = buf[q * CL + cl];
                    s4.x += o.x; s4.y += o.y; s4.z += o.z; s4.w += o.w;
                }
            }
            const float4 u = make_float4(s4.x * inv_n, s4.y * inv_n, s4.z * inv_n, s4.w * inv_n);
            if (UPDATE) {
                if (COMP) {
                    uint32_t b0, b1, b2, b3;
                    float4 ln;
                    two_sum_bf16(v4.x, lo4.x + u.x, vn.x, ln.x, b0);
                    two_sum_bf16(v4.y, lo4.y + u.y, vn.y, ln.y, b1);
                    two_sum_bf16(v4.z, lo4.z + u.z, vn.z, ln.z, b2);
                    two_sum_bf16(v4.w, lo4.w + u.w, vn.w, ln.w, b3);
                    if (!m0) b0 = 0;
                    if (!m1) b1 = 0;
                    if (!m2) b2 = 0;
                    if (!m3) b3 = 0;
                    dv = make_float4((vn.x - v4.x) + (ln.x - lo4.x), (vn.y - v4.y) + (ln.y - lo4.y),
                                     (vn.z - v4.z) + (ln.z - lo4.z), (vn.w - v4.w) + (ln.w - lo4.w));
                    if (rg == 0 && valid) {
                        if (KEEPV) __stcs(reinterpret_cast<uint2*>(lop + col), make_uint2(b0 | (b1 << 16), b2 | (b3 << 16)));
                        else *reinterpret_cast<uint2*>(lop + col) = make_uint2(b0 | (b1 << 16), b2 | (b3 << 16));
                    }
                } else {
                    vn = make_float4(v4.x + u.x, v4.y + u.y, v4.z + u.z, v4.w + u.w);
                    dv = make_float4(vn.x - v4.x, vn.y - v4.y, vn.z - v4.z, vn.w - v4.w);
                }
                if (rg == 0)
                    step_acc += (m0 ? u.x * u.x : 0.f) + (m1 ? u.y * u.y : 0.f) +
                                (m2 ? u.z * u.z : 0.f) + (m3 ? u.w * u.w : 0.f);
            } else {
                vn = u;
            }
        } else if (MODE == PASS_INIT && a.init_mode == BTARD_INIT_ZERO) {
            vn = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (!m0) vn.x = 0.f;
        if (!m1) vn.y = 0.f;
        if (!m2) vn.z = 0.f;
        if (!m3) vn.w = 0.f;
        if (MODE != PASS_NORMS && rg == 0 && valid) {
            if (KEEPV) __stcs(reinterpret_cast<float4*>(vp + col), vn);
            else *reinterpret_cast<float4*>(vp + col) = vn;
        }
        if (MODE == PASS_INIT) dv = vn;                // x still holds the rows themselves

#pragma unroll
        for (int r = 0; r < R; ++r) {                  // residuals at the new v
            const float dx = m0 ? x[r].x - dv.x : 0.f, dy = m1 ? x[r].y - dv.y : 0.f;
            const float dz = m2 ? x[r].z - dv.z : 0.f, dw = m3 ? x[r].w - dv.w : 0.f;
            acc[r] += fmaf(dx, dx, fmaf(dy, dy, fmaf(dz, dz, dw * dw)));
        }
    };

    // Interior tile of an update pass when no row has to be left out: the same update on (column,
    // column + 1) pairs with the packed fp32 instructions of sm_100 (add/sub/mul/fma .f32x2, the IEEE
    // results of two scalar operations each).  d = x - v_hi; s += w d; r = d - e with e = v_lo + (move
    // of v).  The low-order part of v enters the column sums once, as -v_lo * sum_i w_i.
    auto fast_tile = [&](long long qb, int parity) {
        const long long col = (qb + cl) * 4;
        uint64_t xa[R], xb[R];
        const char* xr = reinterpret_cast<const char*>(xrow0 + col);
        if (nrows == R) {                              // the usual case: no row test, no zero fill
#pragma unroll
            for (int r = 0; r < R; ++r, xr += stride_bytes) ld_row_pairs(reinterpret_cast<const float*>(xr), xa[r], xb[r]);
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r, xr += stride_bytes) {
                if (r < nrows) ld_row_pairs(reinterpret_cast<const float*>(xr), xa[r], xb[r]);
                else { xa[r] = 0ull; xb[r] = 0ull; }
            }
        }
        float4 v4;
        asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                     : "=f"(v4.x), "=f"(v4.y), "=f"(v4.z), "=f"(v4.w) : "l"(vp + col), "l"(keep));
        float4 lo4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (COMP) {
            uint2 lb;
            asm volatile("ld.global.L2::cache_hint.v2.u32 {%0, %1}, [%2], %3;" : "=r"(lb.x), "=r"(lb.y) : "l"(lop + col), "l"(keep));
            lo4 = make_float4(bf16_value(lb.x & 0xFFFFu), bf16_value(lb.x >> 16),
                              bf16_value(lb.y & 0xFFFFu), bf16_value(lb.y >> 16));
        }
        const uint64_t va = pack2(v4.x, v4.y), vb = pack2(v4.z, v4.w);
        uint64_t sa = 0ull, sb = 0ull;
        const uint64_t* w2 = reinterpret_cast<const uint64_t*>(sh_w2) + rg * R;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            xa[r] = sub2(xa[r], va);
            xb[r] = sub2(xb[r], vb);
            const uint64_t w = w2[r];
            sa = fma2(w, xa[r], sa);
            sb = fma2(w, xb[r], sb);
        }
        float4 s4;
        unpack2(sa, s4.x, s4.y);
        unpack2(sb, s4.z, s4.w);
        if (RG > 1) {                                  // add the row groups' partial column sums
            float4* buf = sh_x + (size_t)parity * RG * CL;
            buf[rg * CL + cl] = s4;
            __syncthreads();
            s4 = buf[cl];
            for (int q = 1; q < RG; ++q) {
                const float4 o = buf[q * CL + cl];
                s4.x += o.x; s4.y += o.y; s4.z += o.z; s4.w += o.w;
            }
        }
        if (COMP) {
            const float nw = -sh_wsum;
            s4.x = fmaf(nw, lo4.x, s4.x); s4.y = fmaf(nw, lo4.y, s4.y);
            s4.z = fmaf(nw, lo4.z, s4.z); s4.w = fmaf(nw, lo4.w, s4.w);
        }
        const float4 u = make_float4(s4.x * inv_n, s4.y * inv_n, s4.z * inv_n, s4.w * inv_n);
        float4 vn, e4;                                 // new v_hi; v_lo + what the represented v moved by
        if (COMP) {
            uint32_t b0, b1, b2, b3;
            float4 ln;
            two_sum_bf16(v4.x, lo4.x + u.x, vn.x, ln.x, b0);
            two_sum_bf16(v4.y, lo4.y + u.y, vn.y, ln.y, b1);
            two_sum_bf16(v4.z, lo4.z + u.z, vn.z, ln.z, b2);
            two_sum_bf16(v4.w, lo4.w + u.w, vn.w, ln.w, b3);
            e4 = make_float4((vn.x - v4.x) + ln.x, (vn.y - v4.y) + ln.y, (vn.z - v4.z) + ln.z, (vn.w - v4.w) + ln.w);
            if (rg == 0) __stcs(reinterpret_cast<uint2*>(lop + col), make_uint2(b0 | (b1 << 16), b2 | (b3 << 16)));
        } else {
            vn = make_float4(v4.x + u.x, v4.y + u.y, v4.z + u.z, v4.w + u.w);
            e4 = make_float4(vn.x - v4.x, vn.y - v4.y, vn.z - v4.z, vn.w - v4.w);
        }
        if (rg == 0) {
            step_acc += (u.x * u.x + u.y * u.y) + (u.z * u.z + u.w * u.w);
            __stcs(reinterpret_cast<float4*>(vp + col), vn);
        }
        const uint64_t ea = pack2(e4.x, e4.y), eb = pack2(e4.z, e4.w);
#pragma unroll
        for (int r = 0; r < R; ++r) {                  // residuals at the new v
            const uint64_t da = sub2(xa[r], ea), db = sub2(xb[r], eb);
            const uint64_t q2 = fma2(db, db, mul2(da, da));
            float q0f, q1f;
            unpack2(q2, q0f, q1f);
            acc[r] += q0f + q1f;
        }
    };

    for (long long t = 0; t < ntiles; ++t) {
        const long long qb = q0 + (rev ? ntiles - 1 - t : t) * CL;
        const bool inner = (qb + CL <= q1 && qb + CL <= full_quads);
        if (MODE == PASS_ITER) {
            if (inner && !skip_rows && !scaled) fast_tile(qb, (int)(t & 1));
            else tile(std::true_type{}, qb, (int)(t & 1), pol);
        } else {
            if (inner) tile(std::false_type{}, qb, (int)(t & 1), pol);
            else tile(std::true_type{}, qb, (int)(t & 1), pol);
        }
    }

    // CTA reduction: lanes of a warp share a row group, so a warp reduces R rows at once.
    const int warp = tid >> 5, lane = tid & 31, wpg = CL >> 5;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const double s = warp_sum((double)acc[r]);
        if (lane == 0) sh_red[warp][r] = s;
    }
    {
        const double s = warp_sum((double)step_acc);
        if (lane == 0) sh_red[warp][16] = s;
    }
    __syncthreads();
    double* slots = a.slots + (size_t)p * cpp * (n + 1);
    double* dst = slots + (size_t)j * (n + 1);
    for (int i = tid; i <= n; i += blockDim.x) {
        double s = 0.0;
        if (i < n) {
            const int g0 = (i / R) * wpg;
            for (int q = 0; q < wpg; ++q) s += sh_red[g0 + q][i % R];
        } else {
            for (int q = 0; q < wpg; ++q) s += sh_red[q][16];
        }
        dst[i] = s;
    }

    // The CTA that finishes last adds up the partition's slots (fixed grouping, fixed order) and
    // leaves the totals for the next pass.  No CTA waits for another.
    __threadfence();
    __syncthreads();
    if (tid == 0) sh_flag = (atomicAdd(&a.ticket[p], 1u) == (unsigned)(cpp - 1));
    __syncthreads();
    if (!sh_flag) return;
    __threadfence();
    const int per = n + 1;
    int groups = blockDim.x / per;
    if (groups < 1) groups = 1;
    if (groups > cpp) groups = cpp;
    for (int e = tid; e < groups * per; e += blockDim.x) {
        const int cg = e / per, i = e - cg * per;
        double s = 0.0;
        for (int c = cg; c < cpp; c += groups) s += __ldcg(slots + (size_t)c * per + i);
        sh_part[e] = s;
    }
    __syncthreads();
    double* tot = a.tot_out + (size_t)p * per;
    for (int i = tid; i < per; i += blockDim.x) {
        double s = 0.0;
        for (int cg = 0; cg < groups; ++cg) s += sh_part[cg * per + i];
        tot[i] = s;
    }
    if (tid == 0) a.ticket[p] = 0;
}

// =================================================================================================
// Cooperative variant: the start pass and every update of all partitions inside ONE kernel.
//
// The work items are the column ranges the launch-per-update path gives to its CTAs, dealt
// round-robin to one wave of resident CTAs that meet at a grid-wide barrier between updates: no
// launch per update, and nothing runs once the last partition has converged.  The kernel is launched
// cooperatively (the runtime refuses the launch if the CTAs cannot all be resident), every wait on
// the barrier is bounded, and a wait that expires sets an error flag and status bit and makes every
// CTA leave.
// =================================================================================================
struct CoopArgs {
    CclipLaunch a;
    int RG, CL, cppc;               // cppc work items (column ranges) per partition
    int streaming;                  // 1: the tensor is larger than L2 (evict-first loads, alternating sweeps)
    double* rslots;                 // [2][P][cppc][n+1]
    unsigned long long* barrier;    // low word: arrivals (monotonic), high word: finished partitions
    unsigned int* error;            // set when a bounded wait expired
};

constexpr long long kBarrierSpinLimit = 8LL * 1000 * 1000;     // a few seconds of polling

__device__ __forceinline__ unsigned long long ld_volatile_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide barrier.  Returns true when every partition has finished (or a wait ran
// out): the caller then leaves the kernel; CTAs still on their way see the same word and leave too,
// so nobody is left waiting for an arrival that will not come.
__device__ bool grid_barrier(const CoopArgs& k, unsigned& generation, unsigned add_finished, int* sh_flag)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        generation += 1;
        const unsigned long long target = (unsigned long long)generation * gridDim.x;
        const unsigned long long inc = 1ull + ((unsigned long long)add_finished << 32);
        unsigned long long v = atomicAdd(k.barrier, inc) + inc;
        long long spins = 0;
        bool expired = false;
        while ((v & 0xffffffffull) < target && (v >> 32) < (unsigned long long)k.a.P) {
            v = ld_volatile_u64(k.barrier);
            if (++spins > kBarrierSpinLimit) { expired = true; break; }
        }
        if (expired) {
            atomicExch(k.error, 1u);
            atomicAdd(k.barrier, (unsigned long long)k.a.P << 32);   // release everybody else
        }
        if (atomicAdd(k.error, 0u) != 0u) expired = true;
        __threadfence();
        *sh_flag = (expired || (v >> 32) >= (unsigned long long)k.a.P) ? 1 : 0;
    } else {
        generation += 1;
    }
    __syncthreads();
    return *sh_flag != 0;
}

template <int R, bool COMP>
__global__ void __launch_bounds__(512) cclip_cooperative_kernel(const CoopArgs k)
{
    extern __shared__ float4 sh_x[];                  // [2][RG][CL]
    __shared__ double sh_sum[BTARD_MAX_PEERS + 1];
    __shared__ float sh_w[BTARD_MAX_PEERS + 16];
    __shared__ double sh_red[16][17];
    __shared__ double sh_part[512 + BTARD_MAX_PEERS + 1];
    __shared__ int sh_flag, sh_bar;

    const CclipLaunch& a = k.a;
    const int n = a.n, RG = k.RG, CL = k.CL, cppc = k.cppc, Pc = a.P;   // Pc: partitions of this launch
    const int tid = threadIdx.x, cl = tid % CL, rg = tid / CL;
    const int items = Pc * cppc;                       // CTA b owns items b, b + gridDim.x, ...
    const long long stride = a.stride;
    const float inv_n = 1.0f / (float)n;
    const float* wrow = sh_w + rg * R;
    const int per = n + 1;
    const long long Q = stride >> 2;
    const uint64_t policy = policy_evict_first();

    // the work item in hand
    int p = 0, j = 0;
    long long len = 0, q0 = 0, q1 = 0, full_quads = 0, ntiles = 0;
    double tau = 0.0;
    const float* gp = a.g;
    float* vp = a.v;
    unsigned short* lop = nullptr;
    auto take_item = [&](int item) {
        p = item / cppc;
        j = item - p * cppc;
        len = a.table[p].len;
        tau = a.table[p].tau;
        gp = a.g + (size_t)p * n * stride;
        vp = a.v + (size_t)p * stride;
        lop = COMP ? a.v_lo + (size_t)p * stride : nullptr;
        q0 = Q * j / cppc;
        q1 = Q * (j + 1) / cppc;
        if (j > 0) q0 &= ~7LL;
        if (j + 1 < cppc) q1 &= ~7LL;
        full_quads = len >> 2;
        ntiles = (q1 - q0 + CL - 1) / CL;
    };

    float acc[R];
    float step_acc = 0.0f;

    // One tile of CL quads.  INIT: v holds (or becomes) v^0 and the norms at v^0 are taken;
    // otherwise one CenteredClip update.
    auto tile = [&](auto init_tag, auto masked_tag, long long qb, int parity) {
        constexpr bool INIT = decltype(init_tag)::value;
        constexpr bool MASKED = decltype(masked_tag)::value;
        const long long col = (qb + cl) * 4;
        const bool valid = !MASKED || (qb + cl < q1);
        const bool m0 = !MASKED || (valid && col < len), m1 = !MASKED || (valid && col + 1 < len);
        const bool m2 = !MASKED || (valid && col + 2 < len), m3 = !MASKED || (valid && col + 3 < len);
        float4 x[R];
        float4 v4 = make_float4(0.f, 0.f, 0.f, 0.f), lo4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int i = rg * R + r;
                const float* src = gp + (size_t)i * stride + col;
                x[r] = (i >= n) ? make_float4(0.f, 0.f, 0.f, 0.f)
                                : (k.streaming ? ld_policy(src, policy) : __ldg(reinterpret_cast<const float4*>(src)));
            }
            if (!INIT || a.init_mode == BTARD_INIT_CALLER_V0) v4 = *reinterpret_cast<const float4*>(vp + col);
            if (COMP && !INIT) {
                const uint2 lb = *reinterpret_cast<const uint2*>(lop + col);
                lo4 = make_float4(bf16_value(lb.x & 0xFFFFu), bf16_value(lb.x >> 16),
                                  bf16_value(lb.y & 0xFFFFu), bf16_value(lb.y >> 16));
            }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) x[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (!INIT) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                x[r].x = (x[r].x - v4.x) - lo4.x; x[r].y = (x[r].y - v4.y) - lo4.y;
                x[r].z = (x[r].z - v4.z) - lo4.z; x[r].w = (x[r].w - v4.w) - lo4.w;
            }
        }
        float4 vn = v4, dv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!INIT || a.init_mode == BTARD_INIT_MEAN) {
            float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (!INIT) {
                    const float wr = wrow[r];
                    if (wr != 0.0f) {
                        s4.x = fmaf(wr, x[r].x, s4.x); s4.y = fmaf(wr, x[r].y, s4.y);
                        s4.z = fmaf(wr, x[r].z, s4.z); s4.w = fmaf(wr, x[r].w, s4.w);
                    }
                } else {
                    s4.x += x[r].x; s4.y += x[r].y; s4.z += x[r].z; s4.w += x[r].w;
                }
            }
            if (RG > 1) {
                float4* buf = sh_x + (size_t)parity * RG * CL;
                buf[rg * CL + cl] = s4;
                __syncthreads();
                s4 = buf[cl];
                for (int q = 1; q < RG; ++q) {
                    const float4 o = buf[q * CL + cl];
                    s4.x += o.x; s4.y += o.y; s4.z += o.z; s4.w += o.w;
                }
            }
            const float4 u = make_float4(s4.x * inv_n, s4.y * inv_n, s4.z * inv_n, s4.w * inv_n);
            if (!INIT) {
                if (COMP) {
                    uint32_t b0, b1, b2, b3;
                    float4 ln;
                    two_sum_bf16(v4.x, lo4.x + u.x, vn.x, ln.x, b0);
                    two_sum_bf16(v4.y, lo4.y + u.y, vn.y, ln.y, b1);
                    two_sum_bf16(v4.z, lo4.z + u.z, vn.z, ln.z, b2);
                    two_sum_bf16(v4.w, lo4.w + u.w, vn.w, ln.w, b3);
                    if (!m0) b0 = 0;
                    if (!m1) b1 = 0;
                    if (!m2) b2 = 0;
                    if (!m3) b3 = 0;
                    dv = make_float4((vn.x - v4.x) + (ln.x - lo4.x), (vn.y - v4.y) + (ln.y - lo4.y),
                                     (vn.z - v4.z) + (ln.z - lo4.z), (vn.w - v4.w) + (ln.w - lo4.w));
                    if (rg == 0 && valid)
                        *reinterpret_cast<uint2*>(lop + col) = make_uint2(b0 | (b1 << 16), b2 | (b3 << 16));
                } else {
                    vn = make_float4(v4.x + u.x, v4.y + u.y, v4.z + u.z, v4.w + u.w);
                    dv = make_float4(vn.x - v4.x, vn.y - v4.y, vn.z - v4.z, vn.w - v4.w);
                }
                if (rg == 0)
                    step_acc += (m0 ? u.x * u.x : 0.f) + (m1 ? u.y * u.y : 0.f) +
                                (m2 ? u.z * u.z : 0.f) + (m3 ? u.w * u.w : 0.f);
            } else {
                vn = u;
            }
        } else if (INIT && a.init_mode == BTARD_INIT_ZERO) {
            vn = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (!m0) vn.x = 0.f;
        if (!m1) vn.y = 0.f;
        if (!m2) vn.z = 0.f;
        if (!m3) vn.w = 0.f;
        if (rg == 0 && valid) {
            *reinterpret_cast<float4*>(vp + col) = vn;
            if (COMP && INIT) *reinterpret_cast<uint2*>(lop + col) = make_uint2(0u, 0u);
        }
        if (INIT) dv = vn;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float dx = m0 ? x[r].x - dv.x : 0.f, dy = m1 ? x[r].y - dv.y : 0.f;
            const float dz = m2 ? x[r].z - dv.z : 0.f, dw = m3 ? x[r].w - dv.w : 0.f;
            acc[r] += fmaf(dx, dx, fmaf(dy, dy, fmaf(dz, dz, dw * dw)));
        }
    };

    // All tiles of the item in hand, then its partial sums into slot buffer `which`.
    auto sweep = [&](auto init_tag, int which, bool backwards) {
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] = 0.0f;
        step_acc = 0.0f;
        for (long long t = 0; t < ntiles; ++t) {
            const long long qb = q0 + (backwards ? ntiles - 1 - t : t) * CL;
            if (qb + CL <= q1 && qb + CL <= full_quads) tile(init_tag, std::false_type{}, qb, (int)(t & 1));
            else tile(init_tag, std::true_type{}, qb, (int)(t & 1));
        }
        const int warp = tid >> 5, lane = tid & 31, wpg = CL >> 5;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const double s = warp_sum((double)acc[r]);
            if (lane == 0) sh_red[warp][r] = s;
        }
        {
            const double s = warp_sum((double)step_acc);
            if (lane == 0) sh_red[warp][16] = s;
        }
        __syncthreads();
        double* dst = k.rslots + (((size_t)which * Pc + p) * cppc + j) * per;
        for (int i = tid; i <= n; i += blockDim.x) {
            double s = 0.0;
            if (i < n) {
                const int g0 = (i / R) * wpg;
                for (int q = 0; q < wpg; ++q) s += sh_red[g0 + q][i % R];
            } else {
                for (int q = 0; q < wpg; ++q) s += sh_red[q][16];
            }
            dst[i] = s;
        }
    };

    unsigned generation = 0;
    const int first = (int)blockIdx.x, hop = (int)gridDim.x;
    const int mine = first < items ? (items - first + hop - 1) / hop : 0;    // items of this CTA
    for (int m = 0; m < mine; ++m) {
        take_item(first + m * hop);
        if (j == 0 && tid == 0) a.status[p] = 0;
        sweep(std::true_type{}, 0, false);
        __syncthreads();
    }
    if (grid_barrier(k, generation, 0u, &sh_bar)) return;

    const bool eps_mode = (a.stop_mode == BTARD_STOP_EPS);
    for (int l = 0; l <= a.max_iters; ++l) {
        unsigned add_finished = 0;
        // Larger than L2: consecutive updates sweep in opposite directions, so that an update
        // starts on the lines the previous one read last.
        const bool backwards = k.streaming && ((l & 1) == 0);
        for (int m = 0; m < mine; ++m) {
            take_item(first + (backwards ? mine - 1 - m : m) * hop);
            if (a.done[p]) continue;                   // set in an earlier update, behind a barrier
            // Every CTA holding an item of the partition adds up the partition's slots itself, same
            // grouping, same order: identical totals everywhere, nobody waits for a reducer.
            const double* slots = k.rslots + ((size_t)(l & 1) * Pc + p) * cppc * per;
            int groups = blockDim.x / per;
            if (groups < 1) groups = 1;
            if (groups > cppc) groups = cppc;
            for (int e = tid; e < groups * per; e += blockDim.x) {
                const int cg = e / per, i = e - cg * per;
                double s = 0.0;
                for (int c = cg; c < cppc; c += groups) s += __ldcg(slots + (size_t)c * per + i);
                sh_part[e] = s;
            }
            __syncthreads();
            for (int i = tid; i < per; i += blockDim.x) {
                double s = 0.0;
                for (int cg = 0; cg < groups; ++cg) s += sh_part[cg * per + i];
                sh_sum[i] = s;
            }
            if (tid == 0) sh_flag = 0;
            __syncthreads();
            const bool converged = eps_mode && l >= 1 && (sh_sum[n] <= a.eps2);
            if (converged || l == a.max_iters) {
                if (j == 0) {
                    for (int i = tid; i < n; i += blockDim.x) a.resid_norm[(size_t)p * n + i] = sqrt(sh_sum[i]);
                    if (tid == 0) {
                        a.iters[p] = l;
                        a.last_step[p] = sqrt(sh_sum[n]);
                        unsigned st = 0;
                        for (int i = 0; i < n; ++i)
                            if (!isfinite(sh_sum[i])) st |= BTARD_STATUS_NONFINITE_ROW;
                        if (eps_mode && !(sh_sum[n] <= a.eps2)) st |= BTARD_STATUS_NOT_CONVERGED;
                        atomicOr(&a.status[p], st);
                        a.done[p] = 1;                 // read by the other CTAs after the next barrier
                    }
                    add_finished += 1;
                }
            } else {
                const double tau_l = a.tau_sched ? a.tau_sched[(size_t)p * a.max_iters + l] : tau;
                row_weights(sh_sum, sh_w, n, tau_l, a.rule, &sh_flag, sh_part);
                if (j == 0 && tid == 0 && sh_flag) atomicOr(&a.status[p], BTARD_STATUS_NONFINITE_ROW);
                sweep(std::false_type{}, (l + 1) & 1, backwards);
            }
            __syncthreads();                           // shared memory is reused by the next item
        }
        if (grid_barrier(k, generation, add_finished, &sh_bar)) break;
    }
    if (tid == 0 && atomicAdd(k.error, 0u) != 0u)
        for (int m = 0; m < mine; ++m) {
            take_item(first + m * hop);
            if (j == 0) atomicOr(&a.status[p], BTARD_STATUS_WAIT_EXPIRED);
        }
}


// After the last pass: partitions still running take iters = max_iters.
__global__ void cclip_finalize_kernel(const KernelArgs k)
{
    __shared__ double sh_sum[BTARD_MAX_PEERS + 1];
    const CclipLaunch& a = k.a;
    const int p = blockIdx.x, n = a.n;
    if (a.done[p]) return;
    const double* src = a.tot_in + (size_t)p * (n + 1);
    for (int i = threadIdx.x; i <= n; i += blockDim.x) sh_sum[i] = src[i];
    __syncthreads();
    finish_partition(k.a, p, sh_sum, a.max_iters, a.stop_mode == BTARD_STOP_EPS);
}

__global__ void totals_to_norms_kernel(const double* tot, double* norm, int n)
{
    const int p = blockIdx.x;
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        norm[(size_t)p * n + i] = sqrt(tot[(size_t)p * (n + 1) + i]);
}

// ---- coordinate-wise median start ---------------------------------------------------------------
// Order-preserving map of float bit patterns to unsigned integers (IEEE total order).
__device__ __forceinline__ uint32_t order_key_bits(uint32_t u)
{
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t key)
{
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key);
}

// One thread takes the median of the n values of one column.  EXACT: n == N2 is known at compile
// time (the two middle outputs are fixed registers and the network is pruned to them); otherwise
// the column is padded to N2 inputs with the largest value and the middle is picked at run time.
// The kernel is bound by the pipe that executes minimum and maximum, so everything else is kept off
// it: a column whose sum is not NaN holds no NaN and is sorted as floats (no key per input; the sum is
// 64 additions on the other pipe), and with NARROW (row pitch x rows below 4 GiB) the address of row i
// is one wide multiply-add, base + i * pitch, on the multiplier instead of 64-bit additions.  CW = 2
// (exactly 32 or 64 rows): a thread loads two neighbouring columns per row with one address and sorts
// them one after the other.
template <int N2, bool EXACT, bool NARROW, int CW>
__global__ void __launch_bounds__(128, CW == 2 ? 3 : 1) median_sort_kernel(const float* g, float* v,
                                                                           const PartEntry* table, const double* row_scale,
                                                                           long long stride, int n)
{
    __shared__ float sh_f[N2];                         // row factors (with row_scale)
    const int p = blockIdx.y;
    if (row_scale) {
        if (threadIdx.x < N2) sh_f[threadIdx.x] = ((int)threadIdx.x < n) ? (float)row_scale[(size_t)p * n + threadIdx.x] : 0.0f;
        __syncthreads();
    }
    const long long c = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * CW;
    if (c >= stride) return;
    const long long len = table[p].len;
    float out[CW];
#pragma unroll
    for (int w = 0; w < CW; ++w) out[w] = 0.0f;
    if (c < len) {
        const float* gp = g + (size_t)p * n * stride + c;
        const uint32_t pitch = (uint32_t)(stride * 4);     // bytes between rows (NARROW only)
        auto row = [&](int i, float (&o)[CW]) {
            const float* at = gp + (size_t)i * stride;
            if (NARROW) {
                uint64_t a64;
                asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(a64) : "r"((uint32_t)i), "r"(pitch), "l"(gp));
                at = reinterpret_cast<const float*>(a64);
            }
            if constexpr (CW == 2) {
                const float2 t = __ldcs(reinterpret_cast<const float2*>(at));
                o[0] = t.x; o[1] = t.y;
            } else {
                o[0] = __ldcs(at);
            }
        };
        float x[CW][N2];
        float sum[CW][2];
#pragma unroll
        for (int w = 0; w < CW; ++w) sum[w][0] = sum[w][1] = 0.f;
        const float inf = __int_as_float(0x7f800000);      // unused inputs: +infinity
#pragma unroll
        for (int i = 0; i < N2; ++i) {
            float xi[CW];
#pragma unroll
            for (int w = 0; w < CW; ++w) xi[w] = inf;
            if (EXACT || i < n) row(i, xi);
#pragma unroll
            for (int w = 0; w < CW; ++w) x[w][i] = xi[w];
        }
        if (row_scale) {                                   // rows enter as f_i x_i (a factor of 0 reads as zeros)
#pragma unroll
            for (int i = 0; i < N2; ++i) {
                if (EXACT || i < n) {
                    const float f = sh_f[i];
#pragma unroll
                    for (int w = 0; w < CW; ++w) {     // a NaN keeps its own bits (its sign places it in the order)
                        const float xi = x[w][i];
                        x[w][i] = (f == 0.0f) ? 0.0f : (xi == xi) ? f * xi : xi;
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < N2; ++i)
            if (EXACT || i < n) {
#pragma unroll
                for (int w = 0; w < CW; ++w) sum[w][i & 1] += x[w][i];
            }
#pragma unroll
        for (int w = 0; w < CW; ++w) {
            if (w > 0 && c + w >= len) break;
            const float total = sum[w][0] + sum[w][1];
            if (total == total) {                          // no NaN in the column (nor +inf beside -inf)
                out[w] = median_of_values<N2, EXACT>(x[w], n);
            } else {
                int key[N2];
#pragma unroll
                for (int i = 0; i < N2; ++i) key[i] = (EXACT || i < n) ? signed_key(x[w][i]) : 0x7fffffff;
                out[w] = median_of_keys<N2, EXACT>(key, n);
            }
        }
    }
    if constexpr (CW == 2) *reinterpret_cast<float2*>(v + (size_t)p * stride + c) = make_float2(out[0], out[1]);
    else v[(size_t)p * stride + c] = out[0];
}

// The median start and the start pass of the direct algorithm in one read of the rows (exactly 32 or 64
// rows, no row factors): a thread takes the median of a column as above, then reads the column's rows a
// second time (they are in L1: the first read is not marked streaming here) and adds (x_i - v0)^2 to one
// running sum per row.  The sorted copy and the sums are all the registers hold, so the rows are not kept.
// A thread covers at most 512 columns (256 where the slot count allows: fp32 running sums stay short); per-CTA slots and the
// last-CTA reduction are those of the pass kernels, so the first update finds its totals where the start
// pass would have left them.
template <int N2>
__global__ void __launch_bounds__(128, 3) median_norms_kernel(const float* g, float* v, const PartEntry* table,
                                                              long long stride, double* slots_base, double* tot_out,
                                                              unsigned int* ticket, int* done, uint32_t* status,
                                                              long long cols_per_cta)
{
    __shared__ double sh_red[4][N2];
    __shared__ double sh_part[128];
    __shared__ int sh_flag;
    constexpr int n = N2;
    const int p = blockIdx.y, j = blockIdx.x, cpp = gridDim.x, tid = threadIdx.x;
    const long long len = table[p].len;
    if (j == 0 && tid == 0) { done[p] = 0; status[p] = 0; }
    const long long c0 = (long long)j * cols_per_cta;
    long long c1 = c0 + cols_per_cta;
    if (c1 > stride) c1 = stride;
    const float* gp = g + (size_t)p * n * stride;
    const uint32_t pitch = (uint32_t)(stride * 4);         // bytes between rows: the host checked that n rows stay below 4 GiB
    float acc[N2];
#pragma unroll
    for (int i = 0; i < N2; ++i) acc[i] = 0.0f;
    for (long long c = c0 + tid; c < c1; c += 128) {
        float out = 0.0f;
        if (c < len) {
            const float* base = gp + c;
            auto row = [&](int i) {
                uint64_t at;
                asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(at) : "r"((uint32_t)i), "r"(pitch), "l"(base));
                return __ldg(reinterpret_cast<const float*>(at));
            };
            float s[N2];
            float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < N2; ++i) {
                s[i] = row(i);
                sum[i & 3] += s[i];
            }
            const float total = (sum[0] + sum[1]) + (sum[2] + sum[3]);
            if (total == total) {                          // no NaN in the column (nor +inf beside -inf)
                out = median_of_values<N2, true>(s, n);
            } else {
                int key[N2];
#pragma unroll
                for (int i = 0; i < N2; ++i) key[i] = signed_key(s[i]);
                out = median_of_keys<N2, true>(key, n);
            }
#pragma unroll
            for (int i = 0; i < N2; ++i) {
                const float d = row(i) - out;
                acc[i] = fmaf(d, d, acc[i]);
            }
        }
        v[(size_t)p * stride + c] = out;
    }
    // CTA reduction, per-CTA slot, last CTA of the partition adds the slots in a fixed order
    const int warp = tid >> 5, lane = tid & 31;
#pragma unroll
    for (int i = 0; i < N2; ++i) {
        double x = (double)acc[i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
        if (lane == 0) sh_red[warp][i] = x;
    }
    __syncthreads();
    const int per = n + 1;
    double* slots = slots_base + (size_t)p * cpp * per;
    if (tid < per) slots[(size_t)j * per + tid] = (tid < n) ? (sh_red[0][tid] + sh_red[1][tid]) + (sh_red[2][tid] + sh_red[3][tid]) : 0.0;
    __threadfence();
    __syncthreads();
    if (tid == 0) sh_flag = (atomicAdd(&ticket[p], 1u) == (unsigned)(cpp - 1));
    __syncthreads();
    if (!sh_flag) return;
    __threadfence();
    if (tid < per) {
        double t = 0.0;
        for (int c = 0; c < cpp; ++c) t += __ldcg(slots + (size_t)c * per + tid);
        tot_out[(size_t)p * per + tid] = t;
    }
    (void)sh_part;
    if (tid == 0) ticket[p] = 0;
}

// Any n: rank every value by counting (O(n^2) compares per column), pick the two middle ranks.
__global__ void median_rank_kernel(const float* g, float* v, const PartEntry* table, const double* row_scale,
                                   long long stride, int n)
{
    const int p = blockIdx.y;
    const long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= stride) return;
    const long long len = table[p].len;
    float out = 0.0f;
    if (c < len) {
        // The rows are read as bit patterns: the key of a NaN depends on its sign bit, which a floating-point
        // move or product need not keep (with float loads here the key of a positive NaN came out as that of -0).
        const uint32_t* gp = reinterpret_cast<const uint32_t*>(g) + (size_t)p * n * stride + c;
        const int ia = (n - 1) >> 1, ib = n >> 1;
        uint32_t ka = 0, kb = 0;
        const double* fp = row_scale ? row_scale + (size_t)p * n : nullptr;
        auto key_of = [&](int i) {                     // row i as it enters: f_i x_i (a factor of 0 reads as zeros)
            const uint32_t bits = gp[(size_t)i * stride];
            if (fp) {
                const float f = (float)fp[i], x = __uint_as_float(bits);
                if (f == 0.0f) return order_key_bits(0u);
                if (x == x) return order_key_bits(__float_as_uint(f * x));   // a NaN keeps its own bits
            }
            return order_key_bits(bits);
        };
        for (int i = 0; i < n; ++i) {
            const uint32_t ki = key_of(i);
            int rank = 0;
            for (int q = 0; q < n; ++q) {
                const uint32_t kq = key_of(q);
                rank += (kq < ki) || (kq == ki && q < i);
            }
            if (rank == ia) ka = ki;
            if (rank == ib) kb = ki;
        }
        out = (float)(((double)key_value(ka) + (double)key_value(kb)) * 0.5);
    }
    v[(size_t)p * stride + c] = out;
}

template <int R>
int launch_pass_r(const KernelArgs& ka, int mode, int threads, size_t smem, int grid, cudaStream_t st)
{
    const int kind = (mode == PASS_ITER) ? KIND_ITER : (mode == PASS_INIT) ? KIND_INIT
                                              : (mode == PASS_COMBINE) ? KIND_COMBINE : KIND_OTHER;
    prof_begin(kind, st);
    switch (mode) {
        case PASS_INIT: cclip_pass_kernel<R, PASS_INIT, false><<<grid, threads, smem, st>>>(ka); break;
        case PASS_ITER: {
            // programmatic dependent launch: the grid may be set up while the pass before it drains
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3((unsigned)threads);
            cfg.dynamicSmemBytes = smem; cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            cudaError_t e = ka.a.v_lo ? cudaLaunchKernelEx(&cfg, cclip_pass_kernel<R, PASS_ITER, true>, ka)
                                      : cudaLaunchKernelEx(&cfg, cclip_pass_kernel<R, PASS_ITER, false>, ka);
            if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); prof_end(kind, st); return BTARD_ERR_CUDA; }
            break;
        }
        case PASS_COMBINE: cclip_pass_kernel<R, PASS_COMBINE, false><<<grid, threads, smem, st>>>(ka); break;
        default: cclip_pass_kernel<R, PASS_NORMS, false><<<grid, threads, smem, st>>>(ka); break;
    }
    prof_end(kind, st);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

}  // namespace

// Resident CTAs per SM of the iteration kernel for this shape (2 when no device can be asked).
static int iter_ctas_per_sm(int R, int threads, size_t smem)
{
    int nb = 0;
    cudaError_t e;
    if (R == 4) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_pass_kernel<4, PASS_ITER, true>, threads, smem);
    else if (R == 8) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_pass_kernel<8, PASS_ITER, true>, threads, smem);
    else e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_pass_kernel<16, PASS_ITER, true>, threads, smem);
    if (e != cudaSuccess || nb < 1) { (void)cudaGetLastError(); return 2; }
    return nb;
}

// CTAs per partition.  Every CTA pays a fixed cost (its prologue, the first loads, the reduction at
// the end) worth about one and a half tiles of streaming, and a wave of resident CTAs takes as long
// as its longest member, so the estimate to minimise is waves x (tiles per CTA + 1.5), over the counts
// that respect the bound on tiles per CTA.  Measured on n = 16, P = 16, d = 11 M: 18 CTAs per partition
// (one wave, 97 % of the slots) beat 37 (two full waves) by 3.7 %; on n = 64, P = 64, d = 17.7 M: 9
// beat 37 by 8 %, most of it in the passes that find every partition converged.
int choose_ctas_per_partition(int P, long long quads, int CL, int slots, int max_tiles)
{
    const long long tiles = (quads + CL - 1) / CL;
    long long cmin = (tiles + max_tiles - 2) / (max_tiles - 1);
    if (cmin < 1) cmin = 1;
    long long cmax_work = (quads + 7) / 8;             // never less than one 128-byte line per CTA
    if (cmax_work < 1) cmax_work = 1;
    long long lo = cmin, hi = cmin + (4LL * slots + P - 1) / P;
    if (lo > cmax_work) lo = cmax_work;
    if (hi > cmax_work) hi = cmax_work;
    long long best = lo;
    double best_cost = 1e300;
    for (long long c = lo; c <= hi; ++c) {
        const long long total = c * P;
        const long long waves = (total + slots - 1) / slots;
        const double cost = (double)waves * ((double)((tiles + c - 1) / c) + 1.5);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = c; }
    }
    return (int)best;
}

Geometry cclip_geometry(int n, int P, long long stride)
{
    Geometry g;
    g.R = (n <= 4) ? 4 : (n <= 8) ? 8 : 16;
    g.RG = (n + g.R - 1) / g.R;
    g.CL = (g.RG == 1) ? 256 : (g.RG == 2) ? 128 : (g.RG <= 8) ? 64 : 32;
    g.threads = g.RG * g.CL;
    const size_t smem = (g.RG > 1) ? sizeof(float4) * 2 * g.RG * g.CL : 0;
    const int slots = sm_count() * iter_ctas_per_sm(g.R, g.threads, smem);
    g.slots = slots;
    g.cpp = choose_ctas_per_partition(P, stride >> 2, g.CL, slots, kMaxTilesPerPass);
    return g;
}

int launch_cclip_pass(const CclipLaunch& a, const Geometry& geo, int mode, cudaStream_t st)
{
    KernelArgs ka{a, geo.RG, geo.CL, geo.cpp};
    const size_t smem = (geo.RG > 1) ? sizeof(float4) * 2 * geo.RG * geo.CL : 0;
    const int grid = a.P * geo.cpp;
    switch (geo.R) {
        case 4: return launch_pass_r<4>(ka, mode, geo.threads, smem, grid, st);
        case 8: return launch_pass_r<8>(ka, mode, geo.threads, smem, grid, st);
        default: return launch_pass_r<16>(ka, mode, geo.threads, smem, grid, st);
    }
}

int launch_cclip_finalize(const CclipLaunch& a, const Geometry& geo, cudaStream_t st)
{
    KernelArgs ka{a, geo.RG, geo.CL, geo.cpp};
    cclip_finalize_kernel<<<a.P, 128, 0, st>>>(ka);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

int launch_totals_to_norms(const double* tot, double* norm, int n, int P, cudaStream_t st)
{
    totals_to_norms_kernel<<<P, 128, 0, st>>>(tot, norm, n);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

// CTAs per SM of the cooperative kernel (0 when no device can be asked).
static int cooperative_ctas_per_sm(int R, bool comp, int threads, size_t smem)
{
    int nb = 0;
    cudaError_t e;
    if (R == 4) e = comp ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_cooperative_kernel<4, true>, threads, smem)
                         : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_cooperative_kernel<4, false>, threads, smem);
    else if (R == 8) e = comp ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_cooperative_kernel<8, true>, threads, smem)
                              : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_cooperative_kernel<8, false>, threads, smem);
    else e = comp ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_cooperative_kernel<16, true>, threads, smem)
                  : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cclip_cooperative_kernel<16, false>, threads, smem);
    if (e != cudaSuccess || nb < 1) { (void)cudaGetLastError(); return 0; }
    return nb;
}

int launch_cclip_cooperative(const CclipLaunch& a, const Geometry& geo, int streaming, double* rslots,
                             unsigned long long* barrier, unsigned int* error, cudaStream_t st)
{
    CoopArgs ra{a, geo.RG, geo.CL, 0, streaming, rslots, barrier, error};
    const bool comp = a.v_lo != nullptr;
    const size_t smem = (geo.RG > 1) ? sizeof(float4) * 2 * geo.RG * geo.CL : 0;
    const int occ = cooperative_ctas_per_sm(geo.R, comp, geo.threads, smem);
    if (occ < 1) return BTARD_ERR_UNSUPPORTED;
    int grid = sm_count() * occ;
    if (grid > kCoopMaxGrid) grid = kCoopMaxGrid;
    long long cppc = geo.cpp;                          // the work items of the launch-per-update path
    const long long most = ((a.stride >> 2) + 7) / 8;          // at least one 128-byte line per item
    if (cppc > most) cppc = most < 1 ? 1 : most;
    if ((long long)a.P * cppc > kCoopMaxItems) return BTARD_ERR_UNSUPPORTED;
    ra.cppc = (int)cppc;
    if ((long long)grid > (long long)a.P * cppc) grid = (int)((long long)a.P * cppc);
    void* args[] = {(void*)&ra};
    const void* fn;
    if (geo.R == 4) fn = comp ? (const void*)cclip_cooperative_kernel<4, true> : (const void*)cclip_cooperative_kernel<4, false>;
    else if (geo.R == 8) fn = comp ? (const void*)cclip_cooperative_kernel<8, true> : (const void*)cclip_cooperative_kernel<8, false>;
    else fn = comp ? (const void*)cclip_cooperative_kernel<16, true> : (const void*)cclip_cooperative_kernel<16, false>;
    prof_begin(KIND_ITER, st);
    cudaError_t e = cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(geo.threads), args, smem, st);
    prof_end(KIND_ITER, st);
    if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return BTARD_ERR_CUDA; }
    count_launch();
    return BTARD_OK;
}

// 1 when this device can launch cooperative kernels.
int cooperative_launch_supported()
{
    int dev = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return coop;
}

// Whether the fused median + start kernel serves this shape.
bool median_norms_supported(int n, long long stride, const double* row_scale)
{
    // 16 rows: the two separate kernels are both HBM-bound and faster (0.128 + 0.124 against 0.32 ms)
    return (n == 32 || n == 64) && !row_scale && stride * 4 * (long long)n < (1LL << 32);
}

int launch_median_norms(const CclipLaunch& a, const Geometry& geo, cudaStream_t st)
{
    // 256 columns per thread where the slots allow it (the pass kernels' CTAs cover up to 65 536 columns each, so
    // at most 512), enough CTAs for a few waves, and no more CTAs than the slots of the pass kernels hold
    long long cpp = (a.stride + 128LL * 256 - 1) / (128LL * 256);
    const long long want = (4LL * 3 * sm_count() + a.P - 1) / a.P;
    if (cpp < want) cpp = want;
    if (cpp > geo.cpp) cpp = geo.cpp;
    if (cpp < 1) cpp = 1;
    long long cols = (a.stride + cpp - 1) / cpp;
    cols = (cols + 127) / 128 * 128;
    if (cols > 128LL * 512) return BTARD_ERR_UNSUPPORTED;      // cannot happen: geo.cpp bounds the pass kernels' CTAs to 65 536 columns
    cpp = (a.stride + cols - 1) / cols;
    dim3 grid((unsigned)cpp, (unsigned)a.P);
    prof_begin(KIND_MEDIAN, st);
    if (a.n == 64)
        median_norms_kernel<64><<<grid, 128, 0, st>>>(a.g, a.v, a.table, a.stride, a.slots, a.tot_out, a.ticket, a.done, a.status, cols);
    else
        median_norms_kernel<32><<<grid, 128, 0, st>>>(a.g, a.v, a.table, a.stride, a.slots, a.tot_out, a.ticket, a.done, a.status, cols);
    prof_end(KIND_MEDIAN, st);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

int launch_median_init(const float* g, float* v, const PartEntry* table, const double* row_scale,
                       long long stride, int n, int P, cudaStream_t st)
{
    const int threads = 128;
    const int cw = (n == 32 || n == 64) ? 2 : 1;       // two columns per thread: one address per row and pair
    dim3 grid((unsigned)((stride / cw + threads - 1) / threads), (unsigned)P);
    prof_begin(KIND_MEDIAN, st);
    const bool narrow = stride * 4 * (long long)(n > 1 ? n : 1) < (1LL << 32);
#define BTARD_MEDIAN(N2, EX)                                                                              \
    do {                                                                                                  \
        constexpr int CW = (N2 > 16 && EX) ? 2 : 1;                                                           \
        if (narrow) median_sort_kernel<N2, EX, true, CW><<<grid, threads, 0, st>>>(g, v, table, row_scale, stride, n);  \
        else median_sort_kernel<N2, EX, false, CW><<<grid, threads, 0, st>>>(g, v, table, row_scale, stride, n);        \
    } while (0)
    if (n == 1) BTARD_MEDIAN(1, true);
    else if (n == 2) BTARD_MEDIAN(2, true);
    else if (n == 4) BTARD_MEDIAN(4, true);
    else if (n == 8) BTARD_MEDIAN(8, true);
    else if (n == 16) BTARD_MEDIAN(16, true);
    else if (n == 32) BTARD_MEDIAN(32, true);
    else if (n == 64) BTARD_MEDIAN(64, true);
    else if (n < 4) BTARD_MEDIAN(4, false);
    else if (n < 8) BTARD_MEDIAN(8, false);
    else if (n < 16) BTARD_MEDIAN(16, false);
    else if (n < 32) BTARD_MEDIAN(32, false);
    else if (n < 64) BTARD_MEDIAN(64, false);
    else median_rank_kernel<<<grid, threads, 0, st>>>(g, v, table, row_scale, stride, n);
#undef BTARD_MEDIAN
    prof_end(KIND_MEDIAN, st);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

}  // namespace btard
