// Verification pass (Sec. 3.1 eq. (2); Alg. 6, from GetRandomVector to the broadcast of norms and projections) for sm_100a: one read of the
// [P][n][row_stride] tensor produces, per partition, the projections <g_i - v, z_k> on K random
// directions, ||z_k||^2, and the clipped-residual sum sum_i w_i (g_i - v) with its norm.
//
// z is generated on the fly, each quad once per launch.  Up to 16 peers a thread holds every row of
// its 4 columns and draws their z itself (verify_rows_kernel); with more peers the CTA's threads
// share the Philox/Box-Muller work of a [K][tile columns] block of z, stage it in shared memory
// (three buffers), and every thread multiplies its R rows x 4 columns of residuals against it
// (verify_kernel).  Per-thread accumulators are fp32 over at most kMaxTilesPerCta tiles; everything
// that crosses threads is fp64, written to per-CTA slots and summed in a fixed order by the finalize
// kernel.
#include <type_traits>

#include "btard_common.h"
#include "btard_philox.cuh"

namespace btard {
namespace {

__device__ __forceinline__ double warp_sum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    return x;
}

// Streaming 128-bit load of a row's quad as two (column, column + 1) pairs.
__device__ __forceinline__ void ld_stream_pairs(const float* p, uint64_t& lo, uint64_t& hi)
{
    asm volatile("ld.global.cs.v2.b64 {%0, %1}, [%2];" : "=l"(lo), "=l"(hi) : "l"(p));
}

struct VArgs {
    VerifyLaunch a;
    int RG, CL, cpp, slots;
};

// slot layout per CTA: [n*KT] dots (row-major i, k), [KT] znorm2, [1] squared norm of resid_sum
//
// A CTA is RG row groups x CL column lanes; a thread owns R rows x 4 columns of every tile, held as
// (column, column + 1) pairs so that residuals, projections, weighted sums and squared norms run on the
// packed fp32 instructions of sm_100 (two IEEE results per instruction).  The z block of tile t + 1
// is generated during tile t, while the thread's own loads of tile t are in flight, into the third of
// three buffers, so the one CTA barrier per tile hands over what was written a whole tile earlier and
// never waits for the generator.
// COMBINE: as in verify_rows_kernel, the pass first forms v = v0 + sum_j a_j (x_j - v0) from the
// coefficients of the Gram variant.  The row groups' partial moves of v are exchanged through shared
// memory before the same barrier, so the tile loop keeps one barrier.
// Interior tiles (inside the CTA's range and the data, no row to leave out) take a path without any
// predicate; ragged tiles and CTAs with a weight-0 row take the guarded one.
template <int R, int KT, bool COMBINE, int MAXT, int MINB>
__global__ void __launch_bounds__(MAXT, MINB) verify_kernel(const VArgs k)
{
    extern __shared__ float4 sh_dyn[];   // z: [3][KT][CL], column sums: [2][RG][CL], (COMBINE) moves of v: [2][RG][CL]
    __shared__ __align__(8) float2 sh_w2[BTARD_MAX_PEERS + 16];               // (w_i, w_i), zero beyond row n - 1
    __shared__ __align__(8) float2 sh_c2[COMBINE ? BTARD_MAX_PEERS + 16 : 1]; // coefficients (a_j, a_j)
    __shared__ double sh_ga[COMBINE ? BTARD_MAX_PEERS + 1 : 1];               // (G a)_i, then a^T G a
    __shared__ double sh_red[MAXT / 32][R * KT + KT + 1 + (COMBINE ? R : 0)];
    __shared__ float sh_f[BTARD_MAX_PEERS + 16];      // row factors (with row_scale)

    const VerifyLaunch& a = k.a;
    const int n = a.n, RG = k.RG, CL = k.CL, cpp = k.cpp;
    const int tid = threadIdx.x, cl = tid % CL, rg = tid / CL, nthr = blockDim.x;
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const long long stride = a.stride, len = a.table[p].len;
    const double tau = a.table[p].tau;
    float4* sh_z = sh_dyn;
    float4* sh_s = sh_dyn + 3 * KT * CL;
    float4* sh_u = sh_s + 2 * RG * CL;

    const bool scaled = a.row_scale != nullptr;       // rows enter as f_i x_i: applied in the guarded tile path
    for (int i = tid; i < BTARD_MAX_PEERS + 16; i += nthr) {
        sh_w2[i] = make_float2(0.f, 0.f);
        if (COMBINE) sh_c2[i] = make_float2(0.f, 0.f);
        if (scaled) sh_f[i] = (i < n) ? (float)a.row_scale[(size_t)p * n + i] : 0.0f;
    }
    __syncthreads();
    int skip = 0;                                      // some row of this partition must be left out
    if (COMBINE) {
        // clip weights from the Gram matrix: rho_i^2 = G_ii - 2 (G a)_i + a^T G a (rows with a_j = 0 are skipped)
        const double* G = a.gram + (size_t)p * a.gram_entries;
        const double* cf = a.coef + (size_t)p * n;
        for (int i = tid; i < n; i += nthr) {
            double ga = 0.0;
            for (int q = 0; q < n; ++q) {
                const double cq = cf[q];
                if (cq != 0.0) ga += G[gram_entry_index(a.gram_nb, i, q)] * cq;
            }
            sh_ga[i] = ga;
            const float c = (float)cf[i];
            sh_c2[i] = make_float2(c, c);
            if (c == 0.0f) skip = 1;
        }
        __syncthreads();
        if (tid == 0) {
            double aga = 0.0;
            for (int q = 0; q < n; ++q)
                if (cf[q] != 0.0) aga += cf[q] * sh_ga[q];
            sh_ga[n] = aga;
        }
        __syncthreads();
        for (int i = tid; i < n; i += nthr) {
            double rho2 = G[gram_entry_index(a.gram_nb, i, i)] - 2.0 * sh_ga[i] + sh_ga[n];
            if (rho2 < 0.0) rho2 = 0.0;
            const double rho = sqrt(rho2);
            float w = 0.0f;
            if (isfinite(rho)) w = (rho <= tau) ? 1.0f : (float)(tau / rho);
            sh_w2[i] = make_float2(w, w);
            if (w == 0.0f) skip = 1;
        }
    } else {
        for (int i = tid; i < n; i += nthr) {
            const double rho = a.norm_in[(size_t)p * n + i];
            float w = 0.0f;
            if (isfinite(rho)) w = (rho <= tau) ? 1.0f : (float)(tau / rho);
            sh_w2[i] = make_float2(w, w);
            if (w == 0.0f) skip = 1;
        }
    }
    const bool any_skip = __syncthreads_or(skip) != 0;
    const uint64_t* w2 = reinterpret_cast<const uint64_t*>(sh_w2) + rg * R;     // this thread's rows
    const uint64_t* c2 = reinterpret_cast<const uint64_t*>(sh_c2) + (COMBINE ? rg * R : 0);
    unsigned wmask = 0, cmask = 0;                     // rows that enter the weighted sums
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (sh_w2[rg * R + r].x != 0.0f) wmask |= 1u << r;
        if (COMBINE && sh_c2[rg * R + r].x != 0.0f) cmask |= 1u << r;
    }

    // Projections: with few enough of them the sums are kept per (column pair); otherwise one sum
    // per (row, direction) and the two halves of a pair are added on the way in.
    constexpr bool PACC = (2 * R * KT + 4 * R + (COMBINE ? 2 * R : 0) <= ((65536 / (MAXT * MINB) >= 250) ? 200 : (65536 / (MAXT * MINB) >= 160) ? 140 : 72));
    uint64_t acc2[PACC ? R * KT : 1];
    float acc1[PACC ? 1 : R * KT];
#pragma unroll
    for (int e = 0; e < (PACC ? R * KT : 1); ++e) acc2[e] = 0ull;
#pragma unroll
    for (int e = 0; e < (PACC ? 1 : R * KT); ++e) acc1[e] = 0.0f;
    uint64_t nacc2[COMBINE ? R : 1];                   // squared residual norms at the new v
#pragma unroll
    for (int r = 0; r < (COMBINE ? R : 1); ++r) nacc2[r] = 0ull;
    uint64_t zz2[KT];
#pragma unroll
    for (int q = 0; q < KT; ++q) zz2[q] = 0ull;
    float rs2 = 0.0f;

    // This CTA's share of the partition in groups of 4 columns, cut on 128-byte lines.
    const long long Q = stride >> 2;
    long long q0 = Q * j / cpp, q1 = Q * (j + 1) / cpp;
    if (j > 0) q0 &= ~7LL;
    if (j + 1 < cpp) q1 &= ~7LL;
    const long long full_quads = len >> 2;             // quads that lie entirely inside the data
    const float* xrow0 = a.g + ((size_t)p * n + (size_t)rg * R) * stride;   // this thread's first row
    const long long stride_bytes = stride * 4;
    const int nrows = (n - rg * R < R) ? n - rg * R : R;                    // rows of this group that exist
    const float* vp = a.v + (size_t)p * stride;
    float* rsp = a.resid_sum ? a.resid_sum + (size_t)p * stride : nullptr;
    const bool first_chunk = (a.k0 == 0);          // the residual sum is produced once, not per chunk
    const uint32_t pg = (uint32_t)(a.p_base + p);

    // The block of z of the tile that starts at quad qb, into buffer `zbuf` (0..2).  A thread draws
    // the quads of its own column lane: directions rg, rg + RG, ... (the column tests are made once).
    auto gen_z = [&](long long qb, int zbuf) {
        float4* zb = sh_z + (size_t)zbuf * KT * CL + cl;
        const long long quad = qb + cl, col = quad * 4;
        const bool inside = quad < q1 && col < len;
        const bool ragged = col + 3 >= len;            // only the last quad of a ragged partition
        for (int kq = rg; kq < KT; kq += RG) {
            float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            if (inside && kq < a.kc) {
                z = z_quad((uint32_t)quad, pg, (uint32_t)(a.k0 + kq), a.seed_lo, a.seed_hi);
                if (ragged) {
                    if (col + 1 >= len) z.y = 0.f;
                    if (col + 2 >= len) z.z = 0.f;
                    z.w = 0.f;
                }
            }
            zb[kq * CL] = z;
        }
    };
    // Adds up the row groups' column sums of the tile at quad qb (written one tile earlier).
    auto consume_sums = [&](long long qb, int par) {
        if (rg != 0) return;
        if (qb + cl >= q1) return;
        const long long col = (qb + cl) * 4;
        const float4* buf = sh_s + (size_t)par * RG * CL;
        float4 s4 = buf[cl];
        for (int q = 1; q < RG; ++q) {
            const float4 o = buf[q * CL + cl];
            s4.x += o.x; s4.y += o.y; s4.z += o.z; s4.w += o.w;
        }
        rs2 += fmaf(s4.x, s4.x, fmaf(s4.y, s4.y, fmaf(s4.z, s4.z, s4.w * s4.w)));
        if (rsp) *reinterpret_cast<float4*>(rsp + col) = s4;
    };

    // One tile.  GUARD = false: every lane's quad lies inside the CTA's range and the data, and no row
    // has to be left out, so nothing is predicated.
    auto tile = [&](auto guard_tag, long long qb, int par, int zcur) {
        constexpr bool GUARD = decltype(guard_tag)::value;
        const long long col = (qb + cl) * 4;
        const bool valid = !GUARD || (qb + cl < q1);
        uint64_t xa[R], xb[R];                         // columns (0, 1) and (2, 3) of the thread's rows
        uint64_t va = 0ull, vb = 0ull;
        if (valid) {
#pragma unroll
            for (int r = 0; r < R; ++r) { xa[r] = 0ull; xb[r] = 0ull; }
            const char* xr = reinterpret_cast<const char*>(xrow0 + col);      // row rg R, then one stride per row
            if (nrows == R) {
#pragma unroll
                for (int r = 0; r < R; ++r, xr += stride_bytes) ld_stream_pairs(reinterpret_cast<const float*>(xr), xa[r], xb[r]);
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r, xr += stride_bytes)
                    if (r < nrows) ld_stream_pairs(reinterpret_cast<const float*>(xr), xa[r], xb[r]);
            }
            if (GUARD && scaled) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float x0, x1, x2, x3;
                    upk2(xa[r], x0, x1);
                    upk2(xb[r], x2, x3);
                    const float4 y = scale_row(make_float4(x0, x1, x2, x3), sh_f[rg * R + r]);
                    xa[r] = pk2(y.x, y.y);
                    xb[r] = pk2(y.z, y.w);
                }
            }
            const float4 v4 = *reinterpret_cast<const float4*>(vp + col);
            va = pk2(v4.x, v4.y);
            vb = pk2(v4.z, v4.w);
            if (GUARD && col + 3 >= len) {             // what lies beyond the data counts as 0, in the rows and in v
                const bool m0 = col < len, m1 = col + 1 < len, m2 = col + 2 < len;
                va = pk2(m0 ? v4.x : 0.f, m1 ? v4.y : 0.f);
                vb = pk2(m2 ? v4.z : 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float x0, x1, x2, x3;
                    upk2(xa[r], x0, x1);
                    upk2(xb[r], x2, x3);
                    xa[r] = pk2(m0 ? x0 : 0.f, m1 ? x1 : 0.f);
                    xb[r] = pk2(m2 ? x2 : 0.f, 0.f);
                }
            }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) { xa[r] = 0ull; xb[r] = 0ull; }
        }
        // the next tile's z, while the rows of this one are on their way; read after the next barrier
        if (qb + CL < q1) gen_z(qb + CL, zcur == 2 ? 0 : zcur + 1);
        if (COMBINE) {
            // residuals at v0 and this row group's share of the move of v, published before the barrier
            uint64_t ua = 0ull, ub = 0ull;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                xa[r] = pk_sub(xa[r], va);
                xb[r] = pk_sub(xb[r], vb);
                if (!GUARD || ((cmask >> r) & 1u)) {   // coefficient 0: the row is left out, not multiplied
                    const uint64_t c = c2[r];
                    ua = pk_fma(c, xa[r], ua);
                    ub = pk_fma(c, xb[r], ub);
                }
            }
            float4 u;
            upk2(ua, u.x, u.y);
            upk2(ub, u.z, u.w);
            sh_u[(size_t)par * RG * CL + rg * CL + cl] = u;
        }
        __syncthreads();
        if (first_chunk && qb > q0) consume_sums(qb - CL, par ^ 1);

        if (COMBINE) {
            const float4* ubuf = sh_u + (size_t)par * RG * CL;
            float4 u = ubuf[cl];
            for (int q = 1; q < RG; ++q) {
                const float4 o = ubuf[q * CL + cl];
                u.x += o.x; u.y += o.y; u.z += o.z; u.w += o.w;
            }
            float v0x, v0y, v0z, v0w;
            upk2(va, v0x, v0y);
            upk2(vb, v0z, v0w);
            const float4 vn = make_float4(v0x + u.x, v0y + u.y, v0z + u.z, v0w + u.w);
            // what v really moved by (the rounded difference)
            const uint64_t da = pk2(vn.x - v0x, vn.y - v0y), db = pk2(vn.z - v0z, vn.w - v0w);
            if (rg == 0 && valid) *reinterpret_cast<float4*>(a.v_out + (size_t)p * stride + col) = vn;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                xa[r] = pk_sub(xa[r], da);
                xb[r] = pk_sub(xb[r], db);
                nacc2[r] = pk_fma(xb[r], xb[r], pk_fma(xa[r], xa[r], nacc2[r]));
            }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                xa[r] = pk_sub(xa[r], va);
                xb[r] = pk_sub(xb[r], vb);
            }
        }
        // projections
        const float4* zb = sh_z + (size_t)zcur * KT * CL;
#pragma unroll
        for (int q = 0; q < KT; ++q) {
            const float4 z = zb[q * CL + cl];
            const uint64_t za = pk2(z.x, z.y), zc = pk2(z.z, z.w);
            if (rg == 0) zz2[q] = pk_fma(zc, zc, pk_fma(za, za, zz2[q]));
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (PACC) {
                    acc2[r * KT + q] = pk_fma(xb[r], zc, pk_fma(xa[r], za, acc2[r * KT + q]));
                } else {
                    float lo, hi;
                    upk2(pk_fma(xb[r], zc, pk_mul(xa[r], za)), lo, hi);
                    acc1[r * KT + q] += lo + hi;
                }
            }
        }
        // clipped-residual column sums of this row group
        if (first_chunk) {
            uint64_t sa = 0ull, sb = 0ull;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (!GUARD || ((wmask >> r) & 1u)) {   // weight 0: the row is left out, not multiplied
                    const uint64_t w = w2[r];
                    sa = pk_fma(w, xa[r], sa);
                    sb = pk_fma(w, xb[r], sb);
                }
            }
            float4 s4;
            upk2(sa, s4.x, s4.y);
            upk2(sb, s4.z, s4.w);
            sh_s[(size_t)par * RG * CL + rg * CL + cl] = s4;
        }
    };

    if (q0 < q1) gen_z(q0, 0);                         // made visible by the first tile's barrier
    // interior tiles come first: a run without predicates, then the guarded rest
    long long inner_end = (q1 < full_quads) ? q1 : full_quads;
    if (any_skip || scaled) inner_end = q0;
    int par = 0, zcur = 0;
    long long qb = q0;
    for (; qb + CL <= inner_end; qb += CL, par ^= 1, zcur = (zcur == 2 ? 0 : zcur + 1)) tile(std::false_type{}, qb, par, zcur);
    for (; qb < q1; qb += CL, par ^= 1, zcur = (zcur == 2 ? 0 : zcur + 1)) tile(std::true_type{}, qb, par, zcur);
    __syncthreads();
    if (first_chunk && q1 > q0) consume_sums(q0 + (q1 - q0 - 1) / CL * CL, par ^ 1);

    // CTA reduction
    const int warp = tid >> 5, lane = tid & 31, wpg = CL >> 5;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int q = 0; q < KT; ++q) {
            float d;
            if (PACC) {
                float lo, hi;
                upk2(acc2[r * KT + q], lo, hi);
                d = lo + hi;
            } else {
                d = acc1[r * KT + q];
            }
            const double s = warp_sum((double)d);
            if (lane == 0) sh_red[warp][r * KT + q] = s;
        }
#pragma unroll
    for (int q = 0; q < KT; ++q) {
        float lo, hi;
        upk2(zz2[q], lo, hi);
        const double s = warp_sum((double)lo + (double)hi);
        if (lane == 0) sh_red[warp][R * KT + q] = s;
    }
    {
        const double s = warp_sum((double)rs2);
        if (lane == 0) sh_red[warp][R * KT + KT] = s;
    }
    if (COMBINE) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float lo, hi;
            upk2(nacc2[r], lo, hi);
            const double s = warp_sum((double)lo + (double)hi);
            if (lane == 0) sh_red[warp][R * KT + KT + 1 + r] = s;
        }
    }
    __syncthreads();
    double* dst = a.part_out + ((size_t)p * cpp + j) * k.slots;
    // slot: [n KT] dots, [KT] znorm2, the resid-sum slot, then (COMBINE) [n] squared norms
    const int total = n * KT + KT + 1 + (COMBINE ? n : 0);
    for (int e = tid; e < total; e += nthr) {
        double s = 0.0;
        if (e < n * KT) {
            const int i = e / KT, q = e % KT;
            const int g0 = (i / R) * wpg;
            for (int u = 0; u < wpg; ++u) s += sh_red[g0 + u][(i % R) * KT + q];
        } else if (e < n * KT + KT + 1) {
            const int q = e - n * KT;                  // znorm2 slots, then the resid-sum slot
            for (int u = 0; u < wpg; ++u) s += sh_red[u][R * KT + q];
        } else {
            const int i = e - (n * KT + KT + 1);       // squared norm of row i at the new v
            const int g0 = (i / R) * wpg;
            for (int u = 0; u < wpg; ++u) s += sh_red[g0 + u][R * KT + KT + 1 + (i % R)];
        }
        dst[e] = s;
    }
}

// n <= 16, up to eight directions per launch: one thread holds every row of its 4 columns (R >= n
// rows x 4 columns in registers, as in the CenteredClip passes), so it draws the z quads of those
// columns itself (measured against the shared-z kernel with 4 rows per thread, n = 16, d/P = 698 400,
// P = 16: 0.32 against 0.36 ms at K = 4, 0.50 against 0.52 ms at K = 8; n = 4, K = 8: 0.23 against 0.28).  Each quad of z is still generated exactly once per launch, nothing is staged in
// shared memory and the tile loop has no barrier.  Same per-CTA slot layout as verify_kernel.
// COMBINE: the pass also forms v = v0 + sum_j a_j (x_j - v0) from the coefficients of the Gram variant
// (the combine pass and the verification pass in one read of the rows): v holds v0 on entry, every
// thread rewrites its own 4 columns, and the squared residual norms at the new v are one more set of
// per-row sums (slot entries behind the others).  The clip weights that the clipped-residual sum needs
// before the norms of this pass exist come from the Gram matrix: rho_i^2 = G_ii - 2 (G a)_i + a^T G a.
// CTAs per SM by shape: the sums of 16 rows x 4 or 8 directions need the 255 registers of two CTAs of
// 128 threads; smaller shapes run faster with three or four (measured, K = 4 and 8 at n = 4, 8, 16).
constexpr int rows_min_ctas(int R, int KT)
{
    return (KT <= 2 || R == 16) ? 2 : (R == 8 && KT == 8) ? 3 : 4;
}

template <int R, int KT, bool COMBINE, int CL>
__global__ void __launch_bounds__(CL, rows_min_ctas(R, KT)) verify_rows_kernel(const VArgs k)
{
    __shared__ float sh_w[16];
    __shared__ float sh_c[16];                      // COMBINE: coefficients a_j
    __shared__ double sh_ga[17];                    // COMBINE: (G a)_i, then a^T G a
    __shared__ double sh_red[CL / 32][R * KT + KT + 1 + (COMBINE ? R : 0)];
    __shared__ float sh_f[16];                      // row factors (with row_scale)

    const VerifyLaunch& a = k.a;
    const int n = a.n, cpp = k.cpp;
    const int tid = threadIdx.x;
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const bool scaled = a.row_scale != nullptr;     // rows enter as f_i x_i
    if (scaled && tid < 16) sh_f[tid] = (tid < n) ? (float)a.row_scale[(size_t)p * n + tid] : 0.0f;   // before the barriers below
    const long long stride = a.stride, len = a.table[p].len;
    const double tau = a.table[p].tau;

    if (COMBINE) {
        const double* G = a.gram + (size_t)p * a.gram_entries;
        const double* cf = a.coef + (size_t)p * n;
        if (tid < 16) {
            double ga = 0.0;
            if (tid < n)
                for (int q = 0; q < n; ++q) {
                    const double cq = cf[q];
                    if (cq != 0.0) ga += G[gram_entry_index(a.gram_nb, tid, q)] * cq;   // weight-0 rows are skipped
                }
            sh_ga[tid] = ga;
            sh_c[tid] = (tid < n) ? (float)cf[tid] : 0.0f;
        }
        __syncthreads();
        if (tid == 0) {
            double aga = 0.0;
            for (int q = 0; q < n; ++q)
                if (cf[q] != 0.0) aga += cf[q] * sh_ga[q];
            sh_ga[16] = aga;
        }
        __syncthreads();
        if (tid < 16) {
            float w = 0.0f;
            if (tid < n) {
                double rho2 = G[gram_entry_index(a.gram_nb, tid, tid)] - 2.0 * sh_ga[tid] + sh_ga[16];
                if (rho2 < 0.0) rho2 = 0.0;
                const double rho = sqrt(rho2);
                if (isfinite(rho)) w = (rho <= tau) ? 1.0f : (float)(tau / rho);
            }
            sh_w[tid] = w;
        }
    } else if (tid < 16) {
        float w = 0.0f;
        if (tid < n) {
            const double rho = a.norm_in[(size_t)p * n + tid];
            if (isfinite(rho)) w = (rho <= tau) ? 1.0f : (float)(tau / rho);
        }
        sh_w[tid] = w;
    }
    __syncthreads();

    float nacc[COMBINE ? R : 1];                       // COMBINE: squared residual norms at the new v
#pragma unroll
    for (int r = 0; r < (COMBINE ? R : 1); ++r) nacc[r] = 0.0f;
    float acc[R][KT];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int q = 0; q < KT; ++q) acc[r][q] = 0.0f;
    float zz[KT];
#pragma unroll
    for (int q = 0; q < KT; ++q) zz[q] = 0.0f;
    float rs2 = 0.0f;

    // This CTA's share of the partition in groups of 4 columns, cut on 128-byte lines.
    const long long Q = stride >> 2;
    long long q0 = Q * j / cpp, q1 = Q * (j + 1) / cpp;
    if (j > 0) q0 &= ~7LL;
    if (j + 1 < cpp) q1 &= ~7LL;
    const float* gp = a.g + (size_t)p * n * stride;
    const float* vp = a.v + (size_t)p * stride;
    float* rsp = a.resid_sum ? a.resid_sum + (size_t)p * stride : nullptr;
    const bool first_chunk = (a.k0 == 0);          // the residual sum is produced once, not per chunk
    const uint32_t pg = (uint32_t)(a.p_base + p);

    // a row with weight 0 or coefficient 0 (a non-finite row) is left out of the sums, not multiplied
    bool any_skip = false;
    for (int r = 0; r < n; ++r) any_skip |= (sh_w[r] == 0.0f) || (COMBINE && sh_c[r] == 0.0f);

    // GUARD: the quad reaches past the partition's length, or some row has to be left out
    auto tile = [&](auto guard_tag, auto fullk_tag, long long qb) {
        constexpr bool GUARD = decltype(guard_tag)::value;
        constexpr bool FULLK = decltype(fullk_tag)::value;   // every one of the KT directions is drawn: no test per draw
        const long long col = qb * 4;
        float4 x[R];
#pragma unroll
        for (int r = 0; r < R; ++r)
            x[r] = (r < n) ? __ldcs(reinterpret_cast<const float4*>(gp + (size_t)r * stride + col))
                           : make_float4(0.f, 0.f, 0.f, 0.f);
        if (scaled) {
#pragma unroll
            for (int r = 0; r < R; ++r) x[r] = scale_row(x[r], sh_f[r]);
        }
        const float4 v4 = *reinterpret_cast<const float4*>(vp + col);
        // this thread's quads of z: up to two are drawn while the rows are on their way, further ones
        // one at a time between the sums below (registers)
        constexpr int ZE = (KT <= 2) ? KT : 1;
        const bool m0 = !GUARD || col < len, m1 = !GUARD || col + 1 < len, m2 = !GUARD || col + 2 < len,
                   m3 = !GUARD || col + 3 < len;
        auto draw = [&](int q) {
            float4 zq = make_float4(0.f, 0.f, 0.f, 0.f);
            if ((FULLK || q < a.kc) && m0) {
                zq = z_quad((uint32_t)qb, pg, (uint32_t)(a.k0 + q), a.seed_lo, a.seed_hi);
                if (GUARD && !m3) {                    // only the last quad of a ragged partition
                    if (!m1) zq.y = 0.f;
                    if (!m2) zq.z = 0.f;
                    zq.w = 0.f;
                }
            }
            return zq;
        };
        float4 z[ZE];
#pragma unroll
        for (int q = 0; q < ZE; ++q) z[q] = draw(q);
#pragma unroll
        for (int r = 0; r < R; ++r) {
            x[r].x = m0 ? x[r].x - v4.x : 0.f;
            x[r].y = m1 ? x[r].y - v4.y : 0.f;
            x[r].z = m2 ? x[r].z - v4.z : 0.f;
            x[r].w = m3 ? x[r].w - v4.w : 0.f;
        }
        if (COMBINE) {
            // x holds the residuals at v0: move v by u = sum_j a_j (x_j - v0), then the residuals by what v
            // really moved (the rounded difference), and add up the squared norms at the new v
            float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float cr = sh_c[r];
                if (!GUARD || cr != 0.0f) {
                    u.x = fmaf(cr, x[r].x, u.x); u.y = fmaf(cr, x[r].y, u.y);
                    u.z = fmaf(cr, x[r].z, u.z); u.w = fmaf(cr, x[r].w, u.w);
                }
            }
            const float4 vn = make_float4(v4.x + u.x, v4.y + u.y, v4.z + u.z, v4.w + u.w);
            const float4 dv = make_float4(vn.x - v4.x, vn.y - v4.y, vn.z - v4.z, vn.w - v4.w);
            *reinterpret_cast<float4*>(a.v_out + (size_t)p * stride + col) =
                make_float4(m0 ? vn.x : 0.f, m1 ? vn.y : 0.f, m2 ? vn.z : 0.f, m3 ? vn.w : 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                x[r].x = m0 ? x[r].x - dv.x : 0.f; x[r].y = m1 ? x[r].y - dv.y : 0.f;
                x[r].z = m2 ? x[r].z - dv.z : 0.f; x[r].w = m3 ? x[r].w - dv.w : 0.f;
                nacc[r] += fmaf(x[r].x, x[r].x, fmaf(x[r].y, x[r].y, fmaf(x[r].z, x[r].z, x[r].w * x[r].w)));
            }
        }
        auto project = [&](int q, const float4 zq) {
            zz[q] += fmaf(zq.x, zq.x, fmaf(zq.y, zq.y, fmaf(zq.z, zq.z, zq.w * zq.w)));
#pragma unroll
            for (int r = 0; r < R; ++r)
                acc[r][q] = fmaf(x[r].x, zq.x, fmaf(x[r].y, zq.y, fmaf(x[r].z, zq.z, fmaf(x[r].w, zq.w, acc[r][q]))));
        };
#pragma unroll
        for (int q = 0; q < KT; ++q) project(q, (q < ZE) ? z[q] : draw(q));
        if (first_chunk) {                             // clipped-residual sum of these 4 columns
            float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float wr = sh_w[r];
                if (!GUARD || wr != 0.0f) {
                    s4.x = fmaf(wr, x[r].x, s4.x);
                    s4.y = fmaf(wr, x[r].y, s4.y);
                    s4.z = fmaf(wr, x[r].z, s4.z);
                    s4.w = fmaf(wr, x[r].w, s4.w);
                }
            }
            rs2 += fmaf(s4.x, s4.x, fmaf(s4.y, s4.y, fmaf(s4.z, s4.z, s4.w * s4.w)));
            if (rsp) *reinterpret_cast<float4*>(rsp + col) = s4;
        }
    };
    // a launch that draws all of its KT directions (the usual case) runs its whole tiles without a test per draw:
    // 2-7 % at K = 4 and 8 (n = 4: 0.214 against 0.231 ms, n = 16: 0.443 against 0.453 ms with the norms pass)
    if (KT > 2 && a.kc == KT) {
        for (long long qb = q0 + tid; qb < q1; qb += CL) {
            if (!any_skip && qb * 4 + 3 < len) tile(std::false_type{}, std::true_type{}, qb);
            else tile(std::true_type{}, std::false_type{}, qb);
        }
    } else {
        for (long long qb = q0 + tid; qb < q1; qb += CL) {
            if (!any_skip && qb * 4 + 3 < len) tile(std::false_type{}, std::false_type{}, qb);
            else tile(std::true_type{}, std::false_type{}, qb);
        }
    }

    // CTA reduction
    const int warp = tid >> 5, lane = tid & 31;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int q = 0; q < KT; ++q) {
            const double s = warp_sum((double)acc[r][q]);
            if (lane == 0) sh_red[warp][r * KT + q] = s;
        }
#pragma unroll
    for (int q = 0; q < KT; ++q) {
        const double s = warp_sum((double)zz[q]);
        if (lane == 0) sh_red[warp][R * KT + q] = s;
    }
    {
        const double s = warp_sum((double)rs2);
        if (lane == 0) sh_red[warp][R * KT + KT] = s;
    }
    if (COMBINE) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const double s = warp_sum((double)nacc[r]);
            if (lane == 0) sh_red[warp][R * KT + KT + 1 + r] = s;
        }
    }
    __syncthreads();
    double* dst = a.part_out + ((size_t)p * cpp + j) * k.slots;
    // slot: [n KT] dots, [KT] znorm2, the resid-sum slot, then (COMBINE) [n] squared norms
    const int total = n * KT + KT + 1 + (COMBINE ? n : 0);
    for (int e = tid; e < total; e += CL) {
        const int col = (e < n * KT) ? e : R * KT + (e - n * KT);
        double s = 0.0;
        for (int u = 0; u < CL / 32; ++u) s += sh_red[u][col];
        dst[e] = s;
    }
}

// 41 .. 64 peers, the verification pass fused with the combine pass, one or two directions per launch: the four
// lanes 4k .. 4k + 3 of a warp share 4 columns and hold R = 12 or 16 rows each (lane g: rows R g .. R g + R - 1, R x 4
// columns in registers as in verify_rows_kernel), so what the 64 rows of a column have to add up (the move of
// v, the clipped-residual sum) crosses lanes by two shuffle steps and the tile loop has no CTA barrier and no
// shared-memory staging at all.  Direction q of a launch is drawn by lane q of the group and handed to the
// others by shuffle, so every quad of z is still generated once.  Slot layout as verify_kernel.
constexpr int kLanesThreads = 128;
constexpr int kLanesRows = 64;

// One or two directions per launch.  Measured on 64 x 64 x 276 320, K = 1: 0.91 ms with four CTAs per SM (128
// registers, 80 bytes of spills), 0.96 with three (168 registers), 1.02 for the row-group kernel: the pass waits on
// its loads, and more warps hide more of that; two directions spill 280 bytes at 128 registers and keep three
// CTAs.  At four directions (64 x 64 x 4 194 304) neither four lanes of 16 rows (255 registers, two CTAs: 19.9
// against 19.0 ms) nor eight lanes of 8 rows (26.3 ms) beats the row-group kernel, so it keeps them.
// R rows per lane: 12 (41 .. 48 peers) or 16 (49 .. 64).  Measured against the row-group kernel on 16 x n x 276 320,
// K = 1: n = 48: 0.166 against 0.245 ms, n = 40: 0.233 against 0.235, n = 32 (8 rows per lane): 0.129 against 0.127,
// n = 24: 0.175 against 0.116 (half of the lanes hold no rows): used above 40 peers.
template <int R, int KT>
constexpr int lanes_min_ctas() { return (R == 16 && KT == 2) ? 3 : 4; }

// WHOLE: n == 4 R, every lane has all of its rows (a kernel of its own: the row clamp of the other form costs the
// 64-peer shape 5 % through its registers).
template <int R, int KT, bool COMBINE, bool WHOLE>
__global__ void __launch_bounds__(kLanesThreads, lanes_min_ctas<R, KT>()) verify_lanes_kernel(const VArgs k)
{
    constexpr int G = 4, NR = G * R, CL = kLanesThreads;   // four lanes share a quad
    __shared__ float sh_w[NR];
    __shared__ float sh_c[NR];                      // COMBINE: coefficients a_j
    __shared__ double sh_ga[NR + 1];                // COMBINE: (G a)_i, then a^T G a
    __shared__ double sh_red[CL / 32][NR * KT + KT + 1 + (COMBINE ? NR : 0)];
    __shared__ float sh_f[NR];                      // row factors (with row_scale)

    const VerifyLaunch& a = k.a;
    const int n = a.n, cpp = k.cpp;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = tid & (G - 1), rb = R * g;        // lane of the group, its first row
    const unsigned gmask = ((1u << G) - 1u) << (lane & ~(G - 1));   // the lanes that share this thread's columns
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const bool scaled = a.row_scale != nullptr;     // rows enter as f_i x_i
    if (scaled && tid < NR) sh_f[tid] = (tid < n) ? (float)a.row_scale[(size_t)p * n + tid] : 0.0f;   // before the barriers below
    const long long stride = a.stride, len = a.table[p].len;
    const double tau = a.table[p].tau;

    if (COMBINE) {
        const double* G = a.gram + (size_t)p * a.gram_entries;
        const double* cf = a.coef + (size_t)p * n;
        if (tid < NR) {
            double ga = 0.0;
            if (tid < n)
                for (int q = 0; q < n; ++q) {
                    const double cq = cf[q];
                    if (cq != 0.0) ga += G[gram_entry_index(a.gram_nb, tid, q)] * cq;   // weight-0 rows are skipped
                }
            sh_ga[tid] = ga;
            sh_c[tid] = (tid < n) ? (float)cf[tid] : 0.0f;
        }
        __syncthreads();
        if (tid == 0) {
            double aga = 0.0;
            for (int q = 0; q < n; ++q)
                if (cf[q] != 0.0) aga += cf[q] * sh_ga[q];
            sh_ga[NR] = aga;
        }
        __syncthreads();
        if (tid < NR) {
            float w = 0.0f;
            if (tid < n) {
                double rho2 = G[gram_entry_index(a.gram_nb, tid, tid)] - 2.0 * sh_ga[tid] + sh_ga[NR];
                if (rho2 < 0.0) rho2 = 0.0;
                const double rho = sqrt(rho2);
                if (isfinite(rho)) w = (rho <= tau) ? 1.0f : (float)(tau / rho);
            }
            sh_w[tid] = w;
        }
    } else if (tid < NR) {
        float w = 0.0f;
        if (tid < n) {
            const double rho = a.norm_in[(size_t)p * n + tid];
            if (isfinite(rho)) w = (rho <= tau) ? 1.0f : (float)(tau / rho);
        }
        sh_w[tid] = w;
    }
    __syncthreads();

    float nacc[COMBINE ? R : 1];                       // COMBINE: squared residual norms at the new v
#pragma unroll
    for (int r = 0; r < (COMBINE ? R : 1); ++r) nacc[r] = 0.0f;
    float acc[R][KT];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int q = 0; q < KT; ++q) acc[r][q] = 0.0f;
    float zz[KT];
#pragma unroll
    for (int q = 0; q < KT; ++q) zz[q] = 0.0f;
    float rs2 = 0.0f;

    // This CTA's share of the partition in groups of 4 columns, cut on 128-byte lines.
    const long long Q = stride >> 2;
    long long q0 = Q * j / cpp, q1 = Q * (j + 1) / cpp;
    if (j > 0) q0 &= ~7LL;
    if (j + 1 < cpp) q1 &= ~7LL;
    const float* gp = a.g + ((size_t)p * n + rb) * stride;        // this lane's first row
    const float* vp = a.v + (size_t)p * stride;
    float* rsp = a.resid_sum ? a.resid_sum + (size_t)p * stride : nullptr;
    const bool first_chunk = (a.k0 == 0);          // the residual sum is produced once, not per chunk
    const uint32_t pg = (uint32_t)(a.p_base + p);

    // a row with weight 0 or coefficient 0 (a non-finite row) is left out of the sums, not multiplied
    bool any_skip = false;
    for (int r = 0; r < n; ++r) any_skip |= (sh_w[r] == 0.0f) || (COMBINE && sh_c[r] == 0.0f);
    // Whole tiles run without a test per row: a lane that is short of rows reads the partition's last row in
    // their place (finite there, since no row is left out), and what it adds up for them meets a coefficient and a
    // weight of 0 in the column sums and lands in sums that nobody reads.
    const int rmax = n - 1 - rb;

    auto four_sum = [&](float4& s) {                   // sum over the lanes of the group, every lane gets it
#pragma unroll
        for (int o = 1; o < G; o <<= 1) {
            s.x += __shfl_xor_sync(gmask, s.x, o);
            s.y += __shfl_xor_sync(gmask, s.y, o);
            s.z += __shfl_xor_sync(gmask, s.z, o);
            s.w += __shfl_xor_sync(gmask, s.w, o);
        }
    };

    // GUARD: the quad reaches past the partition's length, or some row is missing or has to be left out
    auto tile = [&](auto guard_tag, long long qb) {
        constexpr bool GUARD = decltype(guard_tag)::value;
        const long long col = qb * 4;
        float4 x[R];
#pragma unroll
        for (int r = 0; r < R; ++r)
            x[r] = !GUARD ? __ldcs(reinterpret_cast<const float4*>(gp + (long long)(WHOLE ? r : min(r, rmax)) * stride + col))
                 : (rb + r < n) ? __ldcs(reinterpret_cast<const float4*>(gp + (size_t)r * stride + col))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
        if (scaled) {
#pragma unroll
            for (int r = 0; r < R; ++r) x[r] = scale_row(x[r], sh_f[rb + r]);
        }
        const float4 v4 = *reinterpret_cast<const float4*>(vp + col);
        const bool m0 = !GUARD || col < len, m1 = !GUARD || col + 1 < len, m2 = !GUARD || col + 2 < len,
                   m3 = !GUARD || col + 3 < len;
        // lane q of the group draws direction q while the rows are on their way
        float4 zmine = make_float4(0.f, 0.f, 0.f, 0.f);
        if (g < KT && g < a.kc && m0) {
            zmine = z_quad((uint32_t)qb, pg, (uint32_t)(a.k0 + g), a.seed_lo, a.seed_hi);
            if (GUARD && !m3) {                        // only the last quad of a ragged partition
                if (!m1) zmine.y = 0.f;
                if (!m2) zmine.z = 0.f;
                zmine.w = 0.f;
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool rp = !GUARD || rb + r < n;
            x[r].x = (m0 && rp) ? x[r].x - v4.x : 0.f;
            x[r].y = (m1 && rp) ? x[r].y - v4.y : 0.f;
            x[r].z = (m2 && rp) ? x[r].z - v4.z : 0.f;
            x[r].w = (m3 && rp) ? x[r].w - v4.w : 0.f;
        }
        if (COMBINE) {
            // x holds the residuals at v0: move v by u = sum_j a_j (x_j - v0) over all 64 rows, then the residuals
            // by what v really moved (the rounded difference), and add up the squared norms at the new v
            float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float cr = sh_c[rb + r];
                if (!GUARD || cr != 0.0f) {
                    u.x = fmaf(cr, x[r].x, u.x); u.y = fmaf(cr, x[r].y, u.y);
                    u.z = fmaf(cr, x[r].z, u.z); u.w = fmaf(cr, x[r].w, u.w);
                }
            }
            four_sum(u);
            const float4 vn = make_float4(v4.x + u.x, v4.y + u.y, v4.z + u.z, v4.w + u.w);
            const float4 dv = make_float4(vn.x - v4.x, vn.y - v4.y, vn.z - v4.z, vn.w - v4.w);
            if (g == 0)
                *reinterpret_cast<float4*>(a.v_out + (size_t)p * stride + col) =
                    make_float4(m0 ? vn.x : 0.f, m1 ? vn.y : 0.f, m2 ? vn.z : 0.f, m3 ? vn.w : 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const bool rp = !GUARD || rb + r < n;
                x[r].x = (m0 && rp) ? x[r].x - dv.x : 0.f; x[r].y = (m1 && rp) ? x[r].y - dv.y : 0.f;
                x[r].z = (m2 && rp) ? x[r].z - dv.z : 0.f; x[r].w = (m3 && rp) ? x[r].w - dv.w : 0.f;
                nacc[r] += fmaf(x[r].x, x[r].x, fmaf(x[r].y, x[r].y, fmaf(x[r].z, x[r].z, x[r].w * x[r].w)));
            }
        }
#pragma unroll
        for (int q = 0; q < KT; ++q) {
            const int src = (lane & ~(G - 1)) | q;     // the lane of the group that drew direction q
            float4 zq;
            zq.x = __shfl_sync(gmask, zmine.x, src);
            zq.y = __shfl_sync(gmask, zmine.y, src);
            zq.z = __shfl_sync(gmask, zmine.z, src);
            zq.w = __shfl_sync(gmask, zmine.w, src);
            if (g == 0) zz[q] += fmaf(zq.x, zq.x, fmaf(zq.y, zq.y, fmaf(zq.z, zq.z, zq.w * zq.w)));
#pragma unroll
            for (int r = 0; r < R; ++r)
                acc[r][q] = fmaf(x[r].x, zq.x, fmaf(x[r].y, zq.y, fmaf(x[r].z, zq.z, fmaf(x[r].w, zq.w, acc[r][q]))));
        }
        if (first_chunk) {                             // clipped-residual sum of these 4 columns
            float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float wr = sh_w[rb + r];
                if (!GUARD || wr != 0.0f) {
                    s4.x = fmaf(wr, x[r].x, s4.x);
                    s4.y = fmaf(wr, x[r].y, s4.y);
                    s4.z = fmaf(wr, x[r].z, s4.z);
                    s4.w = fmaf(wr, x[r].w, s4.w);
                }
            }
            four_sum(s4);
            if (g == 0) {
                rs2 += fmaf(s4.x, s4.x, fmaf(s4.y, s4.y, fmaf(s4.z, s4.z, s4.w * s4.w)));
                if (rsp) *reinterpret_cast<float4*>(rsp + col) = s4;
            }
        }
    };
    for (long long qb = q0 + tid / G; qb < q1; qb += CL / G) {
        if (!any_skip && qb * 4 + 3 < len) tile(std::false_type{}, qb);
        else tile(std::true_type{}, qb);
    }

    // CTA reduction: lanes with the same g hold the same rows
    auto rows_sum = [&](double s) {
#pragma unroll
        for (int o = 16; o >= G; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        return s;
    };
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int q = 0; q < KT; ++q) {
            const double s = rows_sum((double)acc[r][q]);
            if (lane < G) sh_red[warp][(rb + r) * KT + q] = s;
        }
#pragma unroll
    for (int q = 0; q < KT; ++q) {
        const double s = warp_sum((double)zz[q]);
        if (lane == 0) sh_red[warp][NR * KT + q] = s;
    }
    {
        const double s = warp_sum((double)rs2);
        if (lane == 0) sh_red[warp][NR * KT + KT] = s;
    }
    if (COMBINE) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const double s = rows_sum((double)nacc[r]);
            if (lane < G) sh_red[warp][NR * KT + KT + 1 + rb + r] = s;
        }
    }
    __syncthreads();
    double* dst = a.part_out + ((size_t)p * cpp + j) * k.slots;
    // slot: [n KT] dots, [KT] znorm2, the resid-sum slot, then (COMBINE) [n] squared norms
    const int total = n * KT + KT + 1 + (COMBINE ? n : 0);
    for (int e = tid; e < total; e += CL) {
        const int col = (e < n * KT) ? e : NR * KT + (e - n * KT);
        double s = 0.0;
        for (int u = 0; u < CL / 32; ++u) s += sh_red[u][col];
        dst[e] = s;
    }
}

// Sums the CTA slots of a partition in a fixed order and writes the outputs of z indices
// k0 .. k0+kc-1 (and, with the first chunk, the per-row and per-partition values).
__global__ void verify_finalize_kernel(const VArgs k, int KT)
{
    extern __shared__ double sh_v[];     // [slots]
    __shared__ float sh_wf[BTARD_MAX_PEERS];
    const VerifyLaunch& a = k.a;
    const int p = blockIdx.x, n = a.n, K = a.K;
    const int total = n * KT + KT + 1 + (a.combine ? n : 0);
    const double* src = a.part_out + (size_t)p * k.cpp * k.slots;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        double s = 0.0;
        for (int c = 0; c < k.cpp; ++c) s += src[(size_t)c * k.slots + e];
        sh_v[e] = s;
    }
    if (a.combine) __syncthreads();                  // the norms below come from the sums above
    const double tau = a.table[p].tau;
    bool bad = false;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const double rho = a.combine ? sqrt(sh_v[n * KT + KT + 1 + i]) : a.norm_in[(size_t)p * n + i];
        float w = 0.0f;
        if (isfinite(rho)) w = (rho <= tau) ? 1.0f : (float)(tau / rho);
        else bad = true;
        sh_wf[i] = w;
        if (a.k0 == 0) {
            a.norm[(size_t)p * n + i] = rho;
            a.weight[(size_t)p * n + i] = (double)w;
        }
        if (a.combine) a.resid_norm_out[(size_t)p * n + i] = rho;
    }
    if (a.k0 == 0 && threadIdx.x == 0) a.status[p] = 0;
    __syncthreads();
    if (bad) atomicOr(&a.status[p], BTARD_STATUS_NONFINITE_ROW);
    if (a.combine) {                                 // what the aggregation's own last kernel would have reported
        if (bad) atomicOr(&a.cclip_status[p], BTARD_STATUS_NONFINITE_ROW);
        if (threadIdx.x == 0 && a.gram_error && *a.gram_error) atomicOr(&a.cclip_status[p], BTARD_STATUS_WAIT_EXPIRED);
    }
    for (int e = threadIdx.x; e < n * a.kc; e += blockDim.x) {
        const int i = e / a.kc, q = e % a.kc;
        const double d = sh_v[i * KT + q];
        const double zn = sqrt(sh_v[n * KT + q]);
        a.dot[((size_t)p * n + i) * K + a.k0 + q] = d;
        a.s[((size_t)p * n + i) * K + a.k0 + q] =
            (sh_wf[i] == 0.0f || zn == 0.0) ? 0.0 : (double)sh_wf[i] * d / zn;
    }
    for (int q = threadIdx.x; q < a.kc; q += blockDim.x) {
        const double zn = sqrt(sh_v[n * KT + q]);
        double ss = 0.0;
        for (int i = 0; i < n; ++i)
            if (sh_wf[i] != 0.0f && zn != 0.0) ss += (double)sh_wf[i] * sh_v[i * KT + q] / zn;
        a.s_sum[(size_t)p * K + a.k0 + q] = ss;
        a.znorm2[(size_t)p * K + a.k0 + q] = sh_v[n * KT + q];
    }
    if (a.k0 == 0 && threadIdx.x == 0) a.resid_sum_norm[p] = sqrt(sh_v[n * KT + KT]);
}

// Verifications 1-3 on broadcast scalars (Alg. 6, the checks each peer runs on them): one CTA per partition.
__device__ __forceinline__ bool differs(double x, double y, double rel_tol, double abs_tol)
{
    const double scale = fmax(fabs(x), fabs(y));
    return !(fabs(x - y) <= rel_tol * scale + abs_tol);      // NaN anywhere: differs
}

__global__ void checks_kernel(const btard_checks_args a)
{
    __shared__ int sh_votes;
    const int p = blockIdx.x, n = a.n_peers, K = a.n_z;
    if (threadIdx.x == 0) sh_votes = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const double nv = a.norm[(size_t)p * n + i];
        a.norm_mismatch[(size_t)p * n + i] =
            a.norm_reported ? (uint8_t)differs(a.norm_reported[(size_t)p * n + i], nv, a.rel_tol, a.abs_tol) : (uint8_t)0;
        const bool far = nv > a.delta_max[p];
        a.check[(size_t)p * n + i] = (uint8_t)far;
        if (far) atomicAdd(&sh_votes, 1);
    }
    for (int e = threadIdx.x; e < n * K; e += blockDim.x) {
        const size_t at = (size_t)p * n * K + e;
        a.s_mismatch[at] = a.s_reported ? (uint8_t)differs(a.s_reported[at], a.s[at], a.rel_tol, a.abs_tol) : (uint8_t)0;
    }
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const double* sv = a.s_reported ? a.s_reported : a.s;
        double sum = 0.0, mag = 0.0;
        for (int i = 0; i < n; ++i) {
            const double v = sv[((size_t)p * n + i) * K + k];
            sum += v;
            mag += fabs(v);
        }
        a.sum_violation[(size_t)p * K + k] = (uint8_t)(!(fabs(sum) <= a.sum_tol * mag));
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        a.votes[p] = sh_votes;
        a.check_averaging[p] = (uint8_t)(2 * sh_votes > n);
    }
}

__global__ void random_vector_kernel(uint32_t seed_lo, uint32_t seed_hi, uint32_t p, uint32_t kz,
                                     long long len, float* z)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (4 * q >= len) return;
    float4 v = z_quad((uint32_t)q, p, kz, seed_lo, seed_hi);
    if (4 * q + 1 >= len) v.y = 0.f;
    if (4 * q + 2 >= len) v.z = 0.f;
    if (4 * q + 3 >= len) v.w = 0.f;
    *reinterpret_cast<float4*>(z + 4 * q) = v;
}

// Shapes and register budgets of the shared-z kernel.  17 to 64 peers: 16 rows per thread in CTAs of
// 128 or 192 threads; with one or two directions two or three CTAs share an SM (168 registers), with
// four the accumulators need the whole file (255 registers, two CTAs of 128 threads).  More peers: one
// warp-wide lane per row group, up to 512 threads.
template <int R, int KT, int MAXT, int MINB>
const void* verify_fn_of(bool combine)
{
    return combine ? (const void*)verify_kernel<R, KT, true, MAXT, MINB> : (const void*)verify_kernel<R, KT, false, MAXT, MINB>;
}

const void* verify_fn(int R, int KT, bool combine, int threads)
{
    if (R == 16 && threads <= 192) {
        // fused with the combine pass the whole register file pays at every K (K = 1, n = 64: 1.02 against 1.07 ms
        // with 0.6 KB of spills at 168 registers); the plain pass runs best with three CTAs per SM (0.71 against 0.73)
        if (KT == 1) return combine ? (const void*)verify_kernel<16, 1, true, 192, 1> : (const void*)verify_kernel<16, 1, false, 192, 2>;
        if (KT == 2) return combine ? (const void*)verify_kernel<16, 2, true, 192, 1> : (const void*)verify_kernel<16, 2, false, 192, 2>;
        // four directions: 168 registers hold the plain pass (three CTAs of 128 threads per SM); fused with
        // the combine pass it needs the whole file (measured: 17.1 ms against 18.0 ms with spills, n = 64, d = 2^28)
        if (KT == 4) return combine ? (const void*)verify_kernel<16, 4, true, 192, 1> : (const void*)verify_kernel<16, 4, false, 192, 2>;
    } else if (R == 16) {
        if (KT == 1) return verify_fn_of<16, 1, 512, 1>(combine);
        if (KT == 2) return verify_fn_of<16, 2, 512, 1>(combine);
    }
    return nullptr;
}

// Dynamic shared memory of the shared-z kernel: z block [3][KT][CL], column sums [2][RG][CL] and, with
// the combine pass fused in, the moves of v [2][RG][CL], as float4.  At most 112 KB (KT = 8, CL = 256),
// which is above the 48 KB a kernel gets without opting in: every instantiation opts in once per device.
constexpr int kVerifyMaxSmem = 128 * 1024;

void ensure_verify_attrs()
{
    static std::atomic<unsigned long long> attrs_set{0};
    if (!device_needs_setup(attrs_set)) return;
    const int shapes[][3] = {{16, 1, 128}, {16, 2, 128}, {16, 4, 128}, {16, 1, 512}, {16, 2, 512}};
    for (const auto& sh : shapes)
        for (int combine = 0; combine < 2; ++combine)
            (void)cudaFuncSetAttribute(verify_fn(sh[0], sh[1], combine != 0, sh[2]),
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kVerifyMaxSmem);
    (void)cudaGetLastError();                          // no device: the sizing falls back to fixed figures
    mark_device_done(attrs_set);
}

int verify_ctas_per_sm(int R, int KT, bool combine, int threads, size_t smem)
{
    ensure_verify_attrs();                             // the occupancy answer depends on the opt-in
    int nb = 0;
    const void* fn = verify_fn(R, KT, combine, threads);
    if (!fn || cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, threads, smem) != cudaSuccess || nb < 1) {
        (void)cudaGetLastError();
        return 2;
    }
    return nb;
}

// One thread per 4 columns with every row: 256 threads for one or two directions (128 registers), 128
// threads for four or eight, whose sums need most of the register file.
inline int rows_threads(int KT) { return KT <= 2 ? 256 : 128; }

template <int R, int KT>
const void* rows_fn_of(bool combine)
{
    constexpr int CL = (KT <= 2) ? 256 : 128;
    if constexpr (R == 16 && KT == 8) {                // fused with the combine pass this shape spills 2 KB: not built
        return combine ? nullptr : (const void*)verify_rows_kernel<R, KT, false, CL>;
    } else {
        return combine ? (const void*)verify_rows_kernel<R, KT, true, CL> : (const void*)verify_rows_kernel<R, KT, false, CL>;
    }
}

template <int R>
const void* rows_fn_r(int KT, bool combine)
{
    switch (KT) {
        case 1: return rows_fn_of<R, 1>(combine);
        case 2: return rows_fn_of<R, 2>(combine);
        case 4: return rows_fn_of<R, 4>(combine);
        case 8: return rows_fn_of<R, 8>(combine);
        default: return nullptr;
    }
}

const void* rows_fn(int R, int KT, bool combine)
{
    return (R == 4) ? rows_fn_r<4>(KT, combine) : (R == 8) ? rows_fn_r<8>(KT, combine) : rows_fn_r<16>(KT, combine);
}

template <int R, bool WHOLE>
const void* lanes_fn_r(int KT, bool combine)
{
    switch (KT) {
        case 1: return combine ? (const void*)verify_lanes_kernel<R, 1, true, WHOLE> : (const void*)verify_lanes_kernel<R, 1, false, WHOLE>;
        case 2: return combine ? (const void*)verify_lanes_kernel<R, 2, true, WHOLE> : (const void*)verify_lanes_kernel<R, 2, false, WHOLE>;
        default: return nullptr;
    }
}

inline int lanes_rows(int n) { return n <= 48 ? 12 : 16; }

const void* lanes_fn(int n, int KT, bool combine)
{
    const int R = lanes_rows(n);
    if (n == 4 * R) return R == 12 ? lanes_fn_r<12, true>(KT, combine) : lanes_fn_r<16, true>(KT, combine);
    return R == 12 ? lanes_fn_r<12, false>(KT, combine) : lanes_fn_r<16, false>(KT, combine);
}

int lanes_ctas_per_sm(int n, int KT, bool combine)
{
    int nb = 0;
    const void* fn = lanes_fn(n, KT, combine);
    if (!fn || cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, kLanesThreads, 0) != cudaSuccess || nb < 1) {
        (void)cudaGetLastError();
        return 2;
    }
    return nb;
}

int rows_ctas_per_sm(int R, int KT, bool combine)
{
    int nb = 0;
    const void* fn = rows_fn(R, KT, combine);
    if (!fn || cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, rows_threads(KT), 0) != cudaSuccess || nb < 1) {
        (void)cudaGetLastError();
        return 2;
    }
    return nb;
}

}  // namespace

VerifyGeometry verify_geometry(int n, int P, long long stride, int K, bool fused)
{
    VerifyGeometry vg;
    Geometry& g = vg.g;
    int kt = 1;
    while (kt < K && kt < 8) kt <<= 1;
    vg.own_z = (n <= 16) ? 1 : 0;
    if (vg.own_z) {                  // every row of a column in one thread: z drawn in registers
        g.R = (n <= 4) ? 4 : (n <= 8) ? 8 : 16;
        if (g.R == 16 && fused && kt > 4) kt = 4;      // 16 rows x 8 directions + the combine pass: 2 KB of spills
        g.RG = 1;
        g.CL = rows_threads(kt);
        g.threads = g.CL;
        vg.KT = kt;
        g.slots = sm_count() * rows_ctas_per_sm(g.R, kt, fused);
        g.cpp = choose_ctas_per_partition(P, stride >> 2, g.CL, g.slots);
        vg.slots = n * kt + kt + 1 + n;    // room for the squared norms of the fused combine pass
        return vg;
    }
    if (fused && n > 40 && n <= kLanesRows && kt <= 2) {   // fused with the combine pass, 41 .. 64 peers (with fewer, lanes
                                                           // of every four would hold few rows or none), one or two directions:
        vg.own_z = 2;                                      // four lanes share the rows of a column quad
        g.R = lanes_rows(n);
        g.RG = 1;
        g.CL = kLanesThreads;
        g.threads = kLanesThreads;
        vg.KT = kt;
        g.slots = sm_count() * lanes_ctas_per_sm(n, kt, true);
        g.cpp = choose_ctas_per_partition(P, stride >> 2, kLanesThreads / 4, g.slots);
        vg.slots = n * kt + kt + 1 + n;
        return vg;
    }
    // 16 rows per thread: few row groups exchange column sums, and the per-tile bookkeeping of a thread
    // is spread over 64 elements (measured at n = 64, K = 4: 14.5 thread instructions per element against
    // 23.5 with 8 rows per thread)
    g.R = 16;
    g.RG = (n + 15) / 16;
    g.CL = (g.RG == 2 || g.RG == 3) ? 64 : 32;
    if (kt > 4) kt = 4;                   // the accumulators of 4 directions are all the registers hold
    if (g.RG > 4 && kt > 2) kt = 2;       // more than 256 threads: 128 registers per thread
    g.threads = g.RG * g.CL;
    vg.KT = kt;
    const size_t smem = sizeof(float4) * (3 * (size_t)kt * g.CL + 2 * (size_t)g.RG * g.CL);
    const size_t smem_fused = smem + sizeof(float4) * 2 * (size_t)g.RG * g.CL;
    const int slots = sm_count() * verify_ctas_per_sm(g.R, kt, fused, g.threads, fused ? smem_fused : smem);
    g.slots = slots;
    g.cpp = choose_ctas_per_partition(P, stride >> 2, g.CL, slots);
    vg.slots = n * kt + kt + 1 + n;             // room for the squared norms of the fused combine pass
    return vg;
}

int launch_verify(const VerifyLaunch& a, const VerifyGeometry& vg, cudaStream_t st)
{
    const Geometry& g = vg.g;
    VArgs va{a, g.RG, g.CL, g.cpp, vg.slots};
    const size_t smem = sizeof(float4) * (3 * (size_t)vg.KT * g.CL + (a.combine ? 4 : 2) * (size_t)g.RG * g.CL);
    const int grid = a.P * g.cpp;
    if (smem > (size_t)kVerifyMaxSmem) return BTARD_ERR_UNSUPPORTED;
    ensure_verify_attrs();
    int rc;
    {
        const void* fn = vg.own_z == 2 ? lanes_fn(a.n, vg.KT, a.combine != 0)
                       : vg.own_z ? rows_fn(g.R, vg.KT, a.combine != 0) : verify_fn(g.R, vg.KT, a.combine != 0, g.threads);
        if (!fn) return BTARD_ERR_UNSUPPORTED;
        void* args[] = {(void*)&va};
        prof_begin(KIND_VERIFY, st);
        const cudaError_t e = cudaLaunchKernel(fn, dim3((unsigned)grid), dim3((unsigned)g.threads), args,
                                               vg.own_z ? 0 : smem, st);
        prof_end(KIND_VERIFY, st);
        BTARD_CUDA_TRY(e);
        count_launch();
        rc = BTARD_OK;
    }
    if (rc != BTARD_OK) return rc;
    verify_finalize_kernel<<<a.P, 128, sizeof(double) * vg.slots, st>>>(va, vg.KT);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

int launch_checks(const btard_checks_args& a, cudaStream_t st)
{
    checks_kernel<<<a.n_partitions, 128, 0, st>>>(a);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

int launch_random_vector(uint64_t seed, int p, int k, long long len, float* z, cudaStream_t st)
{
    const long long quads = (len + 3) / 4;
    if (quads == 0) return BTARD_OK;
    const int threads = 256;
    random_vector_kernel<<<(unsigned)((quads + threads - 1) / threads), threads, 0, st>>>(
        (uint32_t)seed, (uint32_t)(seed >> 32), (uint32_t)p, (uint32_t)k, len, z);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

}  // namespace btard
