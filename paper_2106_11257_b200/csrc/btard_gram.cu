// Gram-matrix variant of CenteredClip (same fixed-point iteration, App. D.2 eq. (CenteredClip),
// carried out in the n-dimensional space of combination coefficients).
//
// With R_i = x_i - v0 and G = R R^T (n x n), every iterate is v^l = v0 + sum_j a_j R_j and
//     ||x_i - v^l||^2 = G_ii - 2 (G a)_i + a^T G a,
//     a^{l+1} = a^l + (w - W a^l) / n,   w_i = min{1, tau / ||x_i - v^l||},  W = sum_i w_i,
//     ||v^{l+1} - v^l||^2 = da^T G da.
// So the tensor is read once to build G (this file), the iteration runs on n x n numbers in fp64,
// and one more pass forms v = v0 + sum_j a_j R_j (the combine mode of the streaming kernel).
//
// G is a dense contraction over the columns, but a thin one (n <= 128 rows against hundreds of thousands
// of columns read once), and the products of residuals that differ by orders of magnitude (attacked rows)
// must stay accurate to about 1e-6 relative for the subtraction above, which rules out single-pass TF32.
// Three kernels, by n: n <= 16 exact fp32 products with all rows of a column in one thread; 17..64 on the
// tcgen05 tensor cores with a TF32 hi/lo split (three products, one instruction); 65..128 fp32 FMA on
// 8 x 8 register blocks from shared memory.
#include <cuda.h>

#include "btard_common.h"
#include "btard_median.cuh"

namespace btard {
namespace {

struct GArgs {
    GramLaunch a;
    GramGeometry g;
};

constexpr int kGramThreads = 256;
constexpr int kPre = 6;   // float4 registers per thread for the tile in flight

// Upper-triangular block index -> (bi, bj), bi <= bj.
__device__ __forceinline__ void block_coords(int blk, int NB, int& bi, int& bj)
{
    bi = 0;
    int rem = blk;
    while (rem >= NB - bi) { rem -= NB - bi; ++bi; }
    bj = bi + rem;
}

__global__ void __launch_bounds__(kGramThreads) gram_kernel(const GArgs k)
{
    extern __shared__ __align__(16) float sh[];
    __shared__ int sh_last;
    const GramLaunch& a = k.a;
    const int n = a.n, NB = k.g.NB, nblk = k.g.nblk, KG = k.g.KG, NP = k.g.NP, TK = k.g.TK;
    const int CHM = (NP >> 2) - 1, cpp = k.g.cpp, tid = threadIdx.x;   // NP/4 is a power of two
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const long long stride = a.stride, len = a.table[p].len;
    const float* gp = a.g + (size_t)p * n * stride;
    const float* vp = a.v0 + (size_t)p * stride;

    // columns of this CTA, cut on 128-byte lines
    long long c0 = stride * j / cpp, c1 = stride * (j + 1) / cpp;
    if (j > 0) c0 &= ~31LL;
    if (j + 1 < cpp) c1 &= ~31LL;
    const int ntiles = (int)((c1 - c0 + TK - 1) / TK);

    const bool active = tid < nblk * KG;
    const int kg = tid / nblk, blk = tid % nblk;
    int bi = 0, bj = 0;
    if (active) block_coords(blk, NB, bi, bj);

    float* As0 = sh;
    float* As1 = sh + (size_t)TK * NP;
    for (int e = tid; e < 2 * TK * NP; e += kGramThreads) sh[e] = 0.0f;   // pad rows stay zero
    __syncthreads();

    const int q4 = TK >> 2;                 // float4 per row of a tile
    const int nload = n * q4;
    float4 pre[kPre];

    auto load_tile = [&](long long cb) {
#pragma unroll
        for (int m = 0; m < kPre; ++m) {
            const int e = tid + kGramThreads * m;
            float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
            if (e < nload) {
                const int row = e / q4, c4 = e - row * q4;
                const long long col = cb + 4 * c4;
                if (col < c1) {
                    float4 x = __ldcs(reinterpret_cast<const float4*>(gp + (size_t)row * stride + col));
                    if (a.row_scale) x = scale_row(x, (float)a.row_scale[(size_t)p * n + row]);
                    const float4 v = *reinterpret_cast<const float4*>(vp + col);
                    r.x = (col < len) ? x.x - v.x : 0.f;
                    r.y = (col + 1 < len) ? x.y - v.y : 0.f;
                    r.z = (col + 2 < len) ? x.z - v.z : 0.f;
                    r.w = (col + 3 < len) ? x.w - v.w : 0.f;
                }
            }
            pre[m] = r;
        }
    };
    // Transposed store: As[kk][row], with the 16-byte chunks of a k-row permuted (XOR with kk/4) so
    // that the 32 lanes (consecutive kk, same row) do not all hit one bank.
    auto store_tile = [&](float* As) {
#pragma unroll
        for (int m = 0; m < kPre; ++m) {
            const int e = tid + kGramThreads * m;
            if (e < nload) {
                const int row = e / q4, c4 = e - row * q4;
                const int ch = row >> 2, sub = row & 3;
                const int phys = ((ch ^ c4) & CHM) * 4 + sub;     // kk >> 2 == c4 for kk = 4 c4 + q
                float* dst = As + (size_t)(4 * c4) * NP + phys;
                dst[0] = pre[m].x;
                dst[NP] = pre[m].y;
                dst[2 * NP] = pre[m].z;
                dst[3 * NP] = pre[m].w;
            }
        }
    };

    float acc[8][8];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[r][c] = 0.0f;

    if (ntiles > 0) {
        load_tile(c0);
        store_tile(As0);
    }
    __syncthreads();
    for (int t = 0; t < ntiles; ++t) {
        const float* As = (t & 1) ? As1 : As0;
        if (t + 1 < ntiles) load_tile(c0 + (long long)(t + 1) * TK);
        if (active) {
            for (int kk = kg; kk < TK; kk += KG) {
                const float* row = As + (size_t)kk * NP;
                const int s = kk >> 2;
                const float4 i0 = *reinterpret_cast<const float4*>(row + (((2 * bi) ^ s) & CHM) * 4);
                const float4 i1 = *reinterpret_cast<const float4*>(row + (((2 * bi + 1) ^ s) & CHM) * 4);
                const float4 j0 = *reinterpret_cast<const float4*>(row + (((2 * bj) ^ s) & CHM) * 4);
                const float4 j1 = *reinterpret_cast<const float4*>(row + (((2 * bj + 1) ^ s) & CHM) * 4);
                const float ai[8] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
                const float aj[8] = {j0.x, j0.y, j0.z, j0.w, j1.x, j1.y, j1.z, j1.w};
#pragma unroll
                for (int r = 0; r < 8; ++r)
#pragma unroll
                    for (int c = 0; c < 8; ++c) acc[r][c] = fmaf(ai[r], aj[c], acc[r][c]);
            }
        }
        if (t + 1 < ntiles) store_tile((t & 1) ? As0 : As1);
        __syncthreads();
    }

    // Add the column groups' partial blocks in fp64, fixed order, through shared memory.
    float* scratch = sh;                                  // [64][256]
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) scratch[(r * 8 + c) * kGramThreads + tid] = active ? acc[r][c] : 0.0f;
    __syncthreads();
    const int entries = k.g.entries;
    double* slots = a.slots + (size_t)p * cpp * entries;
    double* dst = slots + (size_t)j * entries;
    for (int idx = tid; idx < entries; idx += kGramThreads) {
        const int b = idx >> 6, e = idx & 63;
        double s = 0.0;
        for (int q = 0; q < KG; ++q) s += (double)scratch[e * kGramThreads + q * nblk + b];
        dst[idx] = s;
    }

    // The CTA that finishes last adds the partition's slots (nobody waits).
    __threadfence();
    __syncthreads();
    if (tid == 0) sh_last = (atomicAdd(&a.ticket[p], 1u) == (unsigned)(cpp - 1));
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    double* out = a.gram + (size_t)p * entries;
    for (int idx = tid; idx < entries; idx += kGramThreads) {
        double s = 0.0;
#pragma unroll 8
        for (int c = 0; c < cpp; ++c) s += __ldcg(slots + (size_t)c * entries + idx);
        out[idx] = s;
    }
    if (tid == 0) a.ticket[p] = 0;
}

// r = hi + lo with hi on the TF32 grid: round to nearest (ties away from zero, as cvt.rna does for finite
// values) by adding half a TF32 unit to the magnitude bits and clearing the 13 low bits; lo = r - hi is
// exact in fp32 and is handed to the tensor core as it is, which reads only its TF32 part (an error of
// 2^-21 |r| at most, of either sign).  Two integer instructions and one subtraction; a NaN stays a NaN in lo.
__device__ __forceinline__ void split_tf32(float r, uint32_t& hi, uint32_t& lo)
{
    hi = (__float_as_uint(r) + 0x1000u) & 0xFFFFE000u;
    lo = __float_as_uint(r - __uint_as_float(hi));
}

// ---- n <= 16 on the fp32 pipes: every row of a column pair in one thread ---------------------------
// A thread owns 2 columns of every tile of its CTA.  Its R >= n row values (and v0) of the next
// kRowsStages - 1 tiles are on their way into shared memory as 8-byte asynchronous copies (cp.async; a
// thread reads back only what it copied itself, so a wait on its own copy groups is all the
// synchronisation there is), which keeps about 100 KB per SM in flight without holding registers.  The
// thread forms the residuals of the current tile and adds the R (R + 1) / 2 products per column to fp32
// running sums: 8.5 fused multiply-adds per element at R = 16, exact fp32 products, no splitting.  The
// running sums are short: every kRowsFlushTiles tiles a warp adds its lanes' sums (shuffles) and moves
// the result to fp64 in shared memory.
constexpr int kRowsThreads = 256;
constexpr int kRowsFlushTiles = 64;
constexpr int kRowsStages = 3;
constexpr int kRowsTile = 2 * kRowsThreads;              // columns per tile

template <int R>
__host__ __device__ constexpr int rows_stage_bytes() { return (R + 1) * kRowsTile * 4; }   // R rows and v0

// FULL: n == R, no row predicate anywhere.
// MEDIAN: the centre v0 is the coordinate-wise median of the rows, taken here (the thread holds every row of
// its two columns) and written out, instead of being read: the median start costs no pass of its own.
template <int R, bool FULL, bool MEDIAN>
__global__ void __launch_bounds__(kRowsThreads, 1) gram_rows_kernel(const GArgs k)
{
    constexpr int NP = R * (R + 1) / 2;
    constexpr int STAGE = rows_stage_bytes<R>();
    extern __shared__ __align__(16) unsigned char sh_stage[];          // [kRowsStages][R + 1][kRowsTile] floats
    __shared__ double sh_acc[kRowsThreads / 32][NP];
    __shared__ float sh_f[R];                          // row factors (with row_scale)
    __shared__ int sh_last;
    const GramLaunch& a = k.a;
    const int n = a.n, cpp = k.g.cpp, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const bool scaled = a.row_scale != nullptr;        // rows enter as f_i x_i
    if (scaled) {
        if (tid < R) sh_f[tid] = (tid < n) ? (float)a.row_scale[(size_t)p * n + tid] : 0.0f;
        __syncthreads();
    }
    const long long stride = a.stride, len = a.table[p].len;
    const float* gp = a.g + (size_t)p * n * stride;
    const float* vp = a.v0 + (size_t)p * stride;
    float* vout = MEDIAN ? a.v0_out + (size_t)p * stride : nullptr;
    // columns of this CTA, cut on 128-byte lines
    long long c0 = stride * j / cpp, c1 = stride * (j + 1) / cpp;
    if (j > 0) c0 &= ~31LL;
    if (j + 1 < cpp) c1 &= ~31LL;
    const int ntiles = (int)((c1 - c0 + kRowsTile - 1) / kRowsTile);

    for (int e = lane; e < NP; e += 32) sh_acc[warp][e] = 0.0;
    __syncwarp();
    float acc[NP];
#pragma unroll
    for (int e = 0; e < NP; ++e) acc[e] = 0.0f;

    const uint32_t my_base = (uint32_t)__cvta_generic_to_shared(sh_stage) + 8u * (uint32_t)tid;
    // copies of tile t into stage t % kRowsStages (one group per tile, empty groups keep the count uniform)
    auto issue = [&](int t) {
        const long long col = c0 + (long long)t * kRowsTile + 2 * tid;
        if (t < ntiles && col < c1) {                  // row_stride is a multiple of 4: a pair is in or out whole
            const uint32_t dst = my_base + (uint32_t)(t % kRowsStages) * STAGE;
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (FULL || r < n)
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst + (uint32_t)r * (kRowsTile * 4)),
                                 "l"(gp + (size_t)r * stride + col) : "memory");
            if (!MEDIAN)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst + (uint32_t)R * (kRowsTile * 4)),
                             "l"(vp + col) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto flush = [&]() {
#pragma unroll
        for (int e = 0; e < NP; ++e) {
            float sv = acc[e];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sv += __shfl_down_sync(0xffffffffu, sv, o);
            if (lane == 0) sh_acc[warp][e] += (double)sv;
            acc[e] = 0.0f;
        }
    };

#pragma unroll
    for (int t = 0; t < kRowsStages - 1; ++t) issue(t);
    int since_flush = 0;
    for (int t = 0; t < ntiles; ++t) {
        issue(t + kRowsStages - 1);                    // into the stage this thread emptied one tile ago
        asm volatile("cp.async.wait_group %0;" ::"n"(kRowsStages - 1) : "memory");   // tile t has landed
        const long long col = c0 + (long long)t * kRowsTile + 2 * tid;
        const bool m0 = col < len && col < c1, m1 = col + 1 < len && col < c1;
        const uint32_t src = my_base + (uint32_t)(t % kRowsStages) * STAGE;
        float2 x[R], v2 = make_float2(0.f, 0.f);
        if (!MEDIAN)
            asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v2.x), "=f"(v2.y) : "r"(src + (uint32_t)R * (kRowsTile * 4)) : "memory");
#pragma unroll
        for (int r = 0; r < R; ++r)
            asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(x[r].x), "=f"(x[r].y) : "r"(src + (uint32_t)r * (kRowsTile * 4)) : "memory");
        if (scaled) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float f = sh_f[r];
                x[r].x = (f == 0.0f) ? 0.0f : scale_value(x[r].x, f);
                x[r].y = (f == 0.0f) ? 0.0f : scale_value(x[r].y, f);
            }
        }
        if (MEDIAN) {
            // the centre of these two columns: median of the rows as they enter, one column at a time (the
            // comparator network runs on the integer pipe, next to the products below on the other one)
            if (col < c1) {                            // row_stride is a multiple of 4: the pair is in or out whole
                // exactly 16 rows: a column whose sum is not NaN holds no NaN (nor +inf beside -inf) and is sorted
                // as floats: the order of such floats is the order of their keys, and the key of every input is
                // saved (0.400 against 0.408 ms for the whole aggregation of 16 x 16 x 698 400; with fewer rows
                // than the network has inputs the float path is slower, 0.515 against 0.490 ms at 12 rows)
                constexpr bool FLOATS = FULL && R == 16;
                float2 sa = make_float2(0.f, 0.f), sb = make_float2(0.f, 0.f);
                if (FLOATS) {
#pragma unroll
                    for (int r = 0; r < R; r += 2) {
                        sa.x += x[r].x; sa.y += x[r].y;
                        sb.x += x[r + 1].x; sb.y += x[r + 1].y;
                    }
                }
                auto column_median = [&](auto pick, float total) {
                    if (FLOATS && total == total) {
                        float val[R];
#pragma unroll
                        for (int r = 0; r < R; ++r) val[r] = (FULL || r < n) ? pick(x[r]) : __int_as_float(0x7f800000);
                        return median_of_values<R, FULL>(val, n);
                    }
                    int key[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) key[r] = (FULL || r < n) ? signed_key(pick(x[r])) : 0x7fffffff;
                    return median_of_keys<R, FULL>(key, n);
                };
                v2.x = m0 ? column_median([](const float2& q) { return q.x; }, sa.x + sb.x) : 0.0f;
                v2.y = m1 ? column_median([](const float2& q) { return q.y; }, sa.y + sb.y) : 0.0f;
                *reinterpret_cast<float2*>(vout + col) = v2;   // 0 beyond the data
            }
        }
        // residuals; what was never copied (rows >= n, columns beyond the CTA's range or the data) reads as 0
        if (FULL && c0 + (long long)(t + 1) * kRowsTile <= (len < c1 ? len : c1)) {       // whole tile inside
#pragma unroll
            for (int r = 0; r < R; ++r) { x[r].x -= v2.x; x[r].y -= v2.y; }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                x[r].x = (m0 && (FULL || r < n)) ? x[r].x - v2.x : 0.f;
                x[r].y = (m1 && (FULL || r < n)) ? x[r].y - v2.y : 0.f;
            }
        }
        int e = 0;
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int q = i; q < R; ++q, ++e)
                acc[e] = fmaf(x[i].y, x[q].y, fmaf(x[i].x, x[q].x, acc[e]));
        if (++since_flush == kRowsFlushTiles) { flush(); since_flush = 0; }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    flush();
    __syncthreads();

    // pair (i <= q) sits at i R - i (i - 1) / 2 + (q - i); the slot holds whole 8 x 8 blocks
    const int entries = k.g.entries, NB = k.g.NB;
    double* slots = a.slots + (size_t)p * cpp * entries;
    double* dst = slots + (size_t)j * entries;
    for (int idx = tid; idx < entries; idx += kRowsThreads) {
        const int b = idx >> 6, e = idx & 63;
        int bi, bj;
        block_coords(b, NB, bi, bj);
        int r = 8 * bi + (e >> 3), c = 8 * bj + (e & 7);
        if (r > c) { const int sw = r; r = c; c = sw; }
        double sv = 0.0;
        if (c < R) {
            const int at = r * R - r * (r - 1) / 2 + (c - r);
            for (int w = 0; w < kRowsThreads / 32; ++w) sv += sh_acc[w][at];
        }
        dst[idx] = sv;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) sh_last = (atomicAdd(&a.ticket[p], 1u) == (unsigned)(cpp - 1));
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    double* out = a.gram + (size_t)p * entries;
    for (int idx = tid; idx < entries; idx += kRowsThreads) {
        double sv = 0.0;
#pragma unroll 8
        for (int c = 0; c < cpp; ++c) sv += __ldcg(slots + (size_t)c * entries + idx);
        out[idx] = sv;
    }
    if (tid == 0) a.ticket[p] = 0;
}

// ---- constants and helpers of the tcgen05 kernel below ------------------------------------------
constexpr int kUmmaTileCols = 32;                       // one 128-byte swizzle row of TF32
constexpr int kUmmaTileBytes = 64 * 128;                // 64 rows x 128 bytes
constexpr int kUmmaFlushTiles = 4;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    // K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; descriptor version 1 (sm_100)
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

// ---- 17 <= n <= 64: the Gram block on the 5th-generation tensor cores, work split by warp role ----
// Per 32-column tile of a partition:
//   loader         one thread issues one tensor copy (the partition's n rows x 128 bytes, described by a
//                  2-d tensor map over g) and one bulk copy of v0 into a ring of raw stages; an mbarrier
//                  per stage counts the bytes that landed;
//   4 producer     warp w takes tiles w, w + 4, ...: reads the raw tile, forms R = g - v0, splits every
//     warps        value into TF32 hi + lo and writes a 128-row K-major operand tile [hi rows 0..63; lo
//                  rows 0..63] (128-byte rows, 128-byte swizzle) into its operand stage;
//   issuing warp   one thread issues, per 8-column k-block, ONE tcgen05.mma with M = 128, N = 64:
//                  A = the whole operand tile, B = its hi half, so rows 0..63 of the accumulator gather
//                  hi hi^T and rows 64..127 gather lo hi^T;  G = top + bottom + bottom^T (hi lo^T is the
//                  transpose of lo hi^T) is formed once, in fp64, at the end.
// Stages are handed over through mbarriers only (raw full: bytes landed; raw empty and operand full: one
// arrival of the producer warp that owns the tile; operand empty: a tcgen05.commit); nothing in the loop
// synchronises the CTA.  Tensor-core accumulation truncates, so two accumulators of 64 tensor-memory
// columns alternate every kUmmaFlushTiles tiles: the producer warps (they own the four lane quarters)
// read one back and add it to fp32 sums in registers while the tensor core fills the other.  Every wait
// is bounded in time and also ends when another warp has given up; a CTA that gave up raises the error
// flag, waits (bounded) for its copies in flight and for the tensor core, frees its tensor memory and
// leaves.  Shared-memory traffic (TMA write + read of the raw tile, write of the operand tile, operand
// reads of the tensor core: 57 KB per 8 KB of rows) is what bounds this kernel, not HBM.
constexpr int kWsProducerWarps = 4;
constexpr int kWsIssueWarp = kWsProducerWarps;           // warp index of the MMA issuer
constexpr int kWsLoadWarp = kWsProducerWarps + 1;        // warp index of the loader
constexpr int kWsThreads = 32 * (kWsProducerWarps + 2);
constexpr int kWsOpStages = 4;
constexpr int kWsOpBytes = 2 * kUmmaTileBytes;           // hi tile, then lo tile: 128 rows x 128 bytes
constexpr int kWsRawStages = 5;
constexpr int kWsRawBytes = 65 * 128;                    // 64 rows + v0, 128 bytes each
constexpr int kWsTmemCols = 128;                         // two accumulators of 64 columns
constexpr int kWsSmem = kWsOpStages * kWsOpBytes + kWsRawStages * kWsRawBytes + 1024;
static_assert(kUmmaFlushTiles == kWsProducerWarps, "one tile per producer warp and accumulator group");
static_assert(kWsOpStages >= kWsProducerWarps, "every producer warp needs an operand stage of its own");

// Bounded wait on an mbarrier phase: first a plain test, then try_wait with a suspend-time hint (the
// thread sleeps in hardware until the phase completes or the hint runs out).  The bound is on elapsed
// clock cycles (about two seconds), whatever the hardware makes of the hint.
constexpr long long kWsWaitCycles = 4000000000LL;
__device__ __forceinline__ bool mbar_wait_or_quit(uint32_t bar, uint32_t parity, const volatile int* quit)
{
    uint32_t done;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.b32 %0, 1, 0, p;\n}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    const long long start = clock64();
    for (;;) {
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.b32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
        if (done) return true;
        if ((quit && *quit) || clock64() - start > kWsWaitCycles) return false;
    }
}
// 128-bit shared-memory accesses by 32-bit shared address (the address space is explicit, so these are
// always single 128-bit shared loads and stores)
__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 r;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(addr) : "memory");
    return r;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// ROWS_FULL: n == 64, no row predicate anywhere.
template <bool ROWS_FULL>
__global__ void __launch_bounds__(kWsThreads, 2) gram_umma_ws_kernel(const GArgs k, unsigned int* error,
                                                                      const __grid_constant__ CUtensorMap g_map)
{
    extern __shared__ __align__(1024) unsigned char sh_raw[];
    __shared__ __align__(8) unsigned long long sh_op_full[kWsOpStages], sh_op_empty[kWsOpStages];
    __shared__ __align__(8) unsigned long long sh_raw_full[kWsRawStages], sh_raw_empty[kWsRawStages];
    __shared__ __align__(8) unsigned long long sh_acc_full[2], sh_acc_empty[2], sh_drain;
    __shared__ uint32_t sh_tmem;
    __shared__ int sh_last;
    __shared__ int sh_fail;
    __shared__ float sh_f[64];                         // row factors (with row_scale)
    const GramLaunch& a = k.a;
    const int n = a.n, cpp = k.g.cpp, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const bool scaled = a.row_scale != nullptr;        // rows enter as f_i x_i
    if (scaled && tid < 64) sh_f[tid] = (tid < n) ? (float)a.row_scale[(size_t)p * n + tid] : 0.0f;   // before the CTA barrier below
    const long long stride = a.stride, len = a.table[p].len;
    const float* vp = a.v0 + (size_t)p * stride;
    // The CTAs of a partition take its 32-column tiles round-robin (tile j, j + cpp, ...): resident
    // together, they read neighbouring 128-byte pieces of the same rows, so an open DRAM page is used whole.
    const long long all_tiles = (stride + kUmmaTileCols - 1) / kUmmaTileCols;
    const int ntiles = (int)((all_tiles - j + cpp - 1) / cpp);      // tiles j + m cpp < all_tiles
    const int ngroups = (ntiles + kUmmaFlushTiles - 1) / kUmmaFlushTiles;
    auto tile_col = [&](int t) { return ((long long)j + (long long)t * cpp) * kUmmaTileCols; };

    unsigned char* ops = (unsigned char*)(((uintptr_t)sh_raw + 1023) & ~(uintptr_t)1023);   // operand stages
    unsigned char* raws = ops + kWsOpStages * kWsOpBytes;                                     // raw stages
    for (int e = tid; e < kWsOpStages * kWsOpBytes / 16; e += kWsThreads)
        reinterpret_cast<uint4*>(ops)[e] = make_uint4(0u, 0u, 0u, 0u);       // rows n .. 63 stay zero
    if (tid == 0) {
        for (int s = 0; s < kWsOpStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_op_full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_op_empty[s])));
        }
        for (int s = 0; s < kWsRawStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_raw_full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_raw_empty[s])));
        }
        for (int q = 0; q < 2; ++q) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_acc_full[q])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&sh_acc_empty[q])), "r"(kWsProducerWarps));
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_drain)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        sh_fail = 0;
    }
    if (warp == kWsIssueWarp) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh_tmem)), "r"(kWsTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sh_tmem;
    const volatile int* quit = &sh_fail;

    float sum[64];                                     // producer threads: row 32 warp + lane of the accumulator
#pragma unroll
    for (int q = 0; q < 64; ++q) sum[q] = 0.0f;
    int issued = 0;                                    // loader: tiles whose copies have been issued

    if (warp < kWsProducerWarps) {
        // ---------------- producers: warp w turns tiles w, w + 4, ... into operand tiles, whole tiles ----------------
        // lane = (q, ch): rows q + 4 m (m = 0 .. 15), 16-byte chunk ch of each; eight lanes cover one
        // 128-byte row, so the reads and the swizzled writes are free of bank conflicts
        const int q = lane >> 3, ch = lane & 7;
        const uint32_t raw_lane = (uint32_t)(q * 128 + 16 * ch);
        const uint32_t ops_addr = smem_u32(ops), raws_addr = smem_u32(raws);
        const uint32_t op_even = (uint32_t)(q * 128 + ((ch ^ q) << 4));               // rows 8 u + q
        const uint32_t op_odd = (uint32_t)((q + 4) * 128 + ((ch ^ (q + 4)) << 4));   // rows 8 u + 4 + q
        bool ok = true;
        int next_read = 0;                             // next accumulator group to read back

        auto read_back = [&](int grp) -> bool {
            const int qa = grp & 1;
            if (!mbar_wait_or_quit(smem_u32(&sh_acc_full[qa]), (uint32_t)((grp >> 1) & 1), quit)) return false;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem + ((uint32_t)(32 * warp) << 16) + (uint32_t)(64 * qa);
            uint32_t d[64];
#pragma unroll
            for (int h = 0; h < 4; ++h)                // four loads in flight, one wait
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                    "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                    : "=r"(d[16 * h + 0]), "=r"(d[16 * h + 1]), "=r"(d[16 * h + 2]), "=r"(d[16 * h + 3]),
                      "=r"(d[16 * h + 4]), "=r"(d[16 * h + 5]), "=r"(d[16 * h + 6]), "=r"(d[16 * h + 7]),
                      "=r"(d[16 * h + 8]), "=r"(d[16 * h + 9]), "=r"(d[16 * h + 10]), "=r"(d[16 * h + 11]),
                      "=r"(d[16 * h + 12]), "=r"(d[16 * h + 13]), "=r"(d[16 * h + 14]), "=r"(d[16 * h + 15])
                    : "r"(taddr + 16u * h));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int e = 0; e < 64; ++e) sum[e] += __uint_as_float(d[e]);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh_acc_empty[qa]));
            return true;
        };

        for (int t = warp; t < ntiles && ok; t += kWsProducerWarps) {
            const int rs = t % kWsRawStages;
            if (!mbar_wait_or_quit(smem_u32(&sh_raw_full[rs]), (uint32_t)((t / kWsRawStages) & 1), quit)) { ok = false; break; }
            const int s = t % kWsOpStages, use = t / kWsOpStages;
            if (use > 0) {                             // the tensor core must be done reading this stage
                if (!mbar_wait_or_quit(smem_u32(&sh_op_empty[s]), (uint32_t)((use - 1) & 1), quit)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            }
            const uint32_t raw = raws_addr + (uint32_t)rs * kWsRawBytes + raw_lane;
            const uint32_t hi_tile = ops_addr + (uint32_t)s * kWsOpBytes;
            const float4 v4 = lds128(raws_addr + (uint32_t)rs * kWsRawBytes + 64 * 128 + 16 * ch);
            const long long col = tile_col(t) + 4 * ch;
            const bool inside = col + 3 < len;         // chunk inside the data: no predicates
            const bool m0 = col < len, m1 = col + 1 < len, m2 = col + 2 < len;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float4 x[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int m = 8 * half + i;        // row q + 4 m
                    if (ROWS_FULL || q + 4 * m < n) x[i] = lds128(raw + m * 512);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int m = 8 * half + i;
                    if (ROWS_FULL || q + 4 * m < n) {
                        if (scaled) x[i] = scale_row(x[i], sh_f[q + 4 * m]);
                        float r0 = x[i].x - v4.x, r1 = x[i].y - v4.y, r2 = x[i].z - v4.z, r3 = x[i].w - v4.w;
                        if (!inside) {                 // ragged end: what lies beyond len (stale bytes included) is 0
                            r0 = m0 ? r0 : 0.f; r1 = m1 ? r1 : 0.f; r2 = m2 ? r2 : 0.f; r3 = 0.f;
                        }
                        uint32_t h0, h1, h2, h3, l0, l1, l2, l3;
                        split_tf32(r0, h0, l0); split_tf32(r1, h1, l1); split_tf32(r2, h2, l2); split_tf32(r3, h3, l3);
                        const uint32_t off = (uint32_t)((m >> 1) * 1024) + ((m & 1) ? op_odd : op_even);
                        sts128(hi_tile + off, h0, h1, h2, h3);
                        sts128(hi_tile + kUmmaTileBytes + off, l0, l1, l2, l3);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh_raw_empty[rs]));       // the loader may refill the raw stage
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh_op_full[s]));
            // every producer warp fills one tile of each group of kUmmaFlushTiles; with its tile of a group
            // done, it reads back the groups before it while this one is multiplied
            const int grp = t / kUmmaFlushTiles;
            while (ok && next_read < grp) {
                ok = read_back(next_read);
                ++next_read;
            }
        }
        while (ok && next_read < ngroups) {
            ok = read_back(next_read);
            ++next_read;
        }
        if (!ok) sh_fail = 1;
    } else if (warp == kWsIssueWarp) {
        if (lane == 0) {
            // ---------------- the thread that issues the MMAs ----------------
            // tf32 inputs, fp32 accumulate, K-major A and B, N = 64, M = 128
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t op_base = smem_u32(ops);
            bool ok = true;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int s = t % kWsOpStages, use = t / kWsOpStages;
                const int grp = t / kUmmaFlushTiles, first = (t % kUmmaFlushTiles == 0);
                const uint32_t acc = tmem + (uint32_t)(64 * (grp & 1));
                if (first && grp >= 2)                 // the producers must have read this accumulator back
                    ok = mbar_wait_or_quit(smem_u32(&sh_acc_empty[grp & 1]), (uint32_t)(((grp >> 1) - 1) & 1), quit);
                if (ok) ok = mbar_wait_or_quit(smem_u32(&sh_op_full[s]), (uint32_t)(use & 1), quit);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tile_addr = op_base + (uint32_t)s * kWsOpBytes;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {       // 8 TF32 = 32 bytes per k-block
                    const uint64_t d = umma_desc(tile_addr + 32u * ks);     // A: 128 rows; B: its first 64
                    const uint32_t acc0 = (!first || ks > 0) ? 1u : 0u;
                    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
                                 ::"r"(acc), "l"(d), "l"(d), "r"(idesc), "r"(acc0) : "memory");
                }
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(smem_u32(&sh_op_empty[s])) : "memory");
                if ((t + 1) % kUmmaFlushTiles == 0 || t + 1 == ntiles)
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 ::"r"(smem_u32(&sh_acc_full[grp & 1])) : "memory");
            }
            if (!ok) sh_fail = 1;
        }
    } else {
        // ---------------- loader: one tensor copy (n rows x 128 bytes) and one copy of v0 per tile ----------------
        if (lane == 0) {
            uint64_t pol;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
            bool ok = true;
            for (int t = 0; t < ntiles; ++t) {
                const int rs = t % kWsRawStages, use = t / kWsRawStages;
                if (use > 0) ok = mbar_wait_or_quit(smem_u32(&sh_raw_empty[rs]), (uint32_t)((use - 1) & 1), quit);
                if (!ok) break;
                const long long c = tile_col(t);
                const long long rest = stride - c;
                const unsigned vbytes = (unsigned)(rest < kUmmaTileCols ? rest : kUmmaTileCols) * 4u;   // multiple of 16
                unsigned char* dst = raws + (size_t)rs * kWsRawBytes;
                const uint32_t bar = smem_u32(&sh_raw_full[rs]);
                // the tensor copy always delivers the whole box (columns beyond the row end arrive as zeros)
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((unsigned)n * 128u + vbytes) : "memory");
                asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
                             ::"r"(smem_u32(dst)), "l"(&g_map), "r"((int)c), "r"(p * n), "r"(bar), "l"(pol) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_u32(dst + 64 * 128)), "l"(vp + c), "r"(vbytes), "r"(bar) : "memory");
                issued = t + 1;
            }
            if (!ok) sh_fail = 1;
        }
    }
    __syncwarp();
    __syncthreads();
    const bool failed = sh_fail != 0;
    if (failed) {
        if (warp == kWsLoadWarp && lane == 0) {
            // copies still in flight must land before the shared memory goes away
            for (int t = (issued > kWsRawStages ? issued - kWsRawStages : 0); t < issued; ++t)
                (void)mbar_wait_or_quit(smem_u32(&sh_raw_full[t % kWsRawStages]), (uint32_t)((t / kWsRawStages) & 1), nullptr);
        }
        if (warp == kWsIssueWarp && lane == 0) {
            // and the tensor core must be idle before its memory goes away
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                         ::"r"(smem_u32(&sh_drain)) : "memory");
            (void)mbar_wait_or_quit(smem_u32(&sh_drain), 0u, nullptr);
            atomicExch(error, 1u);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == kWsIssueWarp) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kWsTmemCols));
    }

    // accumulator row 32 warp + lane -> fp64 [128][64] in shared memory (the stages are dead now);
    // G = top + bottom + bottom^T -> this CTA's slot
    double* sh_g = reinterpret_cast<double*>(ops);
    if (warp < kWsProducerWarps) {
        const int i = 32 * warp + lane;
#pragma unroll
        for (int q = 0; q < 64; ++q) sh_g[i * 64 + q] = (double)sum[q];
    }
    __syncthreads();
    const int entries = k.g.entries, NB = k.g.NB;
    double* slots = a.slots + (size_t)p * cpp * entries;
    double* dst = slots + (size_t)j * entries;
    for (int idx = tid; idx < entries; idx += kWsThreads) {
        const int b = idx >> 6, e = idx & 63;
        int bi, bj;
        block_coords(b, NB, bi, bj);
        const int r = 8 * bi + (e >> 3), c = 8 * bj + (e & 7);
        dst[idx] = sh_g[r * 64 + c] + (sh_g[(64 + r) * 64 + c] + sh_g[(64 + c) * 64 + r]);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) sh_last = (atomicAdd(&a.ticket[p], 1u) == (unsigned)(cpp - 1));
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    double* out = a.gram + (size_t)p * entries;
    for (int idx = tid; idx < entries; idx += kWsThreads) {
        double s = 0.0;
#pragma unroll 8
        for (int c = 0; c < cpp; ++c) s += __ldcg(slots + (size_t)c * entries + idx);
        out[idx] = s;
    }
    if (tid == 0) a.ticket[p] = 0;
}

// Sum over the threads of the CTA (fixed order).
__device__ double block_sum(double x, double* red)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    __syncthreads();
    if (lane == 0) red[warp] = x;
    __syncthreads();
    double s = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w];
    return s;
}

// The fixed-point iteration on coefficients, one CTA per partition, fp64.
__global__ void __launch_bounds__(kGramThreads) gram_iterate_kernel(const GArgs k)
{
    extern __shared__ __align__(16) double G[];          // [n][n], then delta[n]
    __shared__ double red[8];
    const GramLaunch& a = k.a;
    const int n = a.n, NB = k.g.NB, nblk = k.g.nblk, tid = threadIdx.x;
    const int p = blockIdx.x;
    double* delta = G + (size_t)n * n;
    const double* src = a.gram + (size_t)p * k.g.entries;
    for (int idx = tid; idx < nblk * 64; idx += blockDim.x) {
        const int b = idx >> 6, e = idx & 63;
        int bi, bj;
        block_coords(b, NB, bi, bj);
        const int i = 8 * bi + (e >> 3), jj = 8 * bj + (e & 7);
        if (i < n && jj < n) {
            const double val = src[idx];
            G[(size_t)i * n + jj] = val;
            if (bi != bj) G[(size_t)jj * n + i] = val;
        }
    }
    __syncthreads();

    const double tau = a.table[p].tau;
    const int i = tid;
    const bool row = i < n;
    const double gii = row ? G[(size_t)i * n + i] : 0.0;
    const bool bad = row && !isfinite(gii);
    double ai = 0.0, Gai = 0.0, step2 = 0.0;
    int iters = 0;
    for (int l = 0; l < a.max_iters; ++l) {
        const double aGa = block_sum((row && !bad) ? ai * Gai : 0.0, red);
        const double tau_l = a.tau_sched ? a.tau_sched[(size_t)p * a.max_iters + l] : tau;   // tau_l of App. D.2
        double w = 0.0;
        if (row && !bad) {
            double rho2 = gii - 2.0 * Gai + aGa;
            if (rho2 < 0.0) rho2 = 0.0;
            const double rho = sqrt(rho2);
            if (isfinite(rho)) w = (rho <= tau_l) ? 1.0 : tau_l / rho;
        }
        const double W = block_sum(w, red);
        const double d = (row && !bad) ? (w - W * ai) / (double)n : 0.0;
        if (row) delta[i] = d;
        __syncthreads();
        double Gd = 0.0;
        if (row && !bad) {
            for (int q = 0; q < n; ++q) {
                const double dq = delta[q];
                if (dq != 0.0) Gd += G[(size_t)q * n + i] * dq;     // G is symmetric: column read
            }
        }
        step2 = block_sum((row && !bad) ? d * Gd : 0.0, red);
        ai += d;
        Gai += Gd;
        iters = l + 1;
        if (a.stop_mode == BTARD_STOP_EPS && step2 <= a.eps2) break;
    }
    if (step2 < 0.0) step2 = 0.0;
    if (row) a.coef[(size_t)p * n + i] = ai;
    const double anybad = block_sum(bad ? 1.0 : 0.0, red);
    if (tid == 0) {
        a.iters[p] = iters;
        a.last_step[p] = sqrt(step2);
        unsigned st = 0;
        if (anybad > 0.0) st |= BTARD_STATUS_NONFINITE_ROW;
        if (a.stop_mode == BTARD_STOP_EPS && !(step2 <= a.eps2)) st |= BTARD_STATUS_NOT_CONVERGED;
        a.status[p] = st;
    }
}

// n <= 32: the same iteration by ONE warp per partition, lane i owning row i of G in registers.
// Sums are butterfly shuffles (every lane gets the same value), so there is no barrier at all and
// an update costs a few hundred cycles instead of six CTA-wide synchronisations.
template <int N>   // 16 or 32: rows of G held per lane
__global__ void __launch_bounds__(32) gram_iterate_warp_kernel(const GArgs k)
{
    const GramLaunch& a = k.a;
    const int n = a.n, NB = k.g.NB, lane = threadIdx.x, p = blockIdx.x;
    // 16 rows live in 16 lanes: the other half of the warp leaves, and every sum is one step shorter
    constexpr unsigned MASK = (N == 16) ? 0x0000ffffu : 0xffffffffu;
    if (N == 16 && lane >= 16) return;
    const double* src = a.gram + (size_t)p * k.g.entries;
    double Grow[N];
    const bool row = lane < n;
#pragma unroll
    for (int jj = 0; jj < N; ++jj) {
        double val = 0.0;
        if (row && jj < n) {
            const int i0 = lane < jj ? lane : jj, j0 = lane < jj ? jj : lane;   // stored triangle: bi <= bj
            const int bi = i0 >> 3, bj = j0 >> 3;
            int blk = bj - bi;
            for (int q = 0; q < bi; ++q) blk += NB - q;
            // inside a diagonal block both orders are stored and equal; elsewhere (i0, j0) is stored
            val = src[(size_t)blk * 64 + (i0 & 7) * 8 + (j0 & 7)];
        }
        Grow[jj] = val;
    }
    const double tau = a.table[p].tau;
    double gii = 0.0;
#pragma unroll
    for (int jj = 0; jj < N; ++jj)
        if (jj == lane) gii = Grow[jj];
    const bool bad = row && !isfinite(gii);
    const bool live = row && !bad;
    // One update is a chain of dependent double-precision operations, so the chain is kept short: one
    // reciprocal square root instead of a square root and a division (tau / rho = tau rsqrt(rho^2)), a
    // multiplication by 1/n, four partial sums, and two rounds of lane-to-lane traffic per update (the weights
    // to every lane, then one butterfly for the two scalars) instead of three.
    const double tau2 = tau * tau, inv_n = 1.0 / (double)n;
    double ai = 0.0, Gai = 0.0, step2 = 0.0;
    double aGa = 0.0;              // a^T G a, carried along: (a + d)^T G (a + d) = a^T G a + 2 d^T G a + d^T G d
    int iters = 0;
    const double* sched = a.tau_sched ? a.tau_sched + (size_t)p * a.max_iters : nullptr;   // tau_l of App. D.2
    for (int l = 0; l < a.max_iters; ++l) {
        const double tau_l = sched ? sched[l] : tau, tau_l2 = sched ? tau_l * tau_l : tau2;
        double w = 0.0;
        if (live) {
            double rho2 = gii - 2.0 * Gai + aGa;
            if (rho2 < 0.0) rho2 = 0.0;
            if (isfinite(rho2)) w = (rho2 <= tau_l2) ? 1.0 : tau_l * rsqrt(rho2);
        }
        // Every lane fetches every weight once and forms both W = sum_q w_q and (G w)_i from them; the
        // update d = (w - W a) / n then needs no sum of its own, and G d = (G w - W G a) / n.
        double part[4] = {0.0, 0.0, 0.0, 0.0}, wsum[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
        for (int q = 0; q < N; ++q) {
            const double wq = __shfl_sync(MASK, w, q);
            wsum[q & 3] += wq;
            if (wq != 0.0 && live) part[q & 3] += Grow[q] * wq;     // weight-0 rows are skipped, not multiplied
        }
        const double W = (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]);
        const double Gw = (part[0] + part[1]) + (part[2] + part[3]);
        const double d = live ? (w - W * ai) * inv_n : 0.0;
        const double Gd = live ? (Gw - W * Gai) * inv_n : 0.0;
        double dGa = live ? d * Gai : 0.0;             // both sums ride the same butterfly
        step2 = live ? d * Gd : 0.0;
#pragma unroll
        for (int o = N / 2; o > 0; o >>= 1) {
            step2 += __shfl_xor_sync(MASK, step2, o);
            dGa += __shfl_xor_sync(MASK, dGa, o);
        }
        aGa += 2.0 * dGa + step2;
        ai += d;
        Gai += Gd;
        iters = l + 1;
        if (a.stop_mode == BTARD_STOP_EPS && step2 <= a.eps2) break;
    }
    if (step2 < 0.0) step2 = 0.0;
    if (row) a.coef[(size_t)p * n + lane] = ai;
    const unsigned anybad = __ballot_sync(MASK, bad);
    if (lane == 0) {
        a.iters[p] = iters;
        a.last_step[p] = sqrt(step2);
        unsigned st = 0;
        if (anybad) st |= BTARD_STATUS_NONFINITE_ROW;
        if (a.stop_mode == BTARD_STOP_EPS && !(step2 <= a.eps2)) st |= BTARD_STATUS_NOT_CONVERGED;
        a.status[p] = st;
    }
}

__global__ void gram_finalize_kernel(const double* tot, double* resid_norm, uint32_t* status, int n,
                                     const unsigned int* error)
{
    const int p = blockIdx.x;
    bool bad = false;
    if (threadIdx.x == 0 && error && *error) atomicOr(&status[p], BTARD_STATUS_WAIT_EXPIRED);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const double v = tot[(size_t)p * (n + 1) + i];
        resid_norm[(size_t)p * n + i] = sqrt(v);
        if (!isfinite(v)) bad = true;
    }
    if (bad) atomicOr(&status[p], BTARD_STATUS_NONFINITE_ROW);
}

// cuTensorMapEncodeTiled, looked up through the runtime so that the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn()
{
    static const EncodeTiledFn fn = [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            ptr = nullptr;
        }
        return (EncodeTiledFn)ptr;
    }();
    return fn;
}

// g [P][n][stride] as a 2-d tensor of P n rows; one box = the n rows of a partition x 32 columns.
bool encode_rows_map(CUtensorMap* map, const float* g, int n, int P, long long stride)
{
    const EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)stride, (cuuint64_t)P * (cuuint64_t)n};
    const cuuint64_t strides[1] = {(cuuint64_t)stride * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)kUmmaTileCols, (cuuint32_t)n};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(g), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// The n <= 16 Gram kernel for R rows per thread (4, 8 or 16), with or without row predicates and median.
static const void* rows_fn(int R, bool full, bool median)
{
    if (R == 4) return full ? (median ? (const void*)gram_rows_kernel<4, true, true> : (const void*)gram_rows_kernel<4, true, false>)
                            : (median ? (const void*)gram_rows_kernel<4, false, true> : (const void*)gram_rows_kernel<4, false, false>);
    if (R == 8) return full ? (median ? (const void*)gram_rows_kernel<8, true, true> : (const void*)gram_rows_kernel<8, true, false>)
                            : (median ? (const void*)gram_rows_kernel<8, false, true> : (const void*)gram_rows_kernel<8, false, false>);
    return full ? (median ? (const void*)gram_rows_kernel<16, true, true> : (const void*)gram_rows_kernel<16, true, false>)
                : (median ? (const void*)gram_rows_kernel<16, false, true> : (const void*)gram_rows_kernel<16, false, false>);
}

GramGeometry gram_geometry(int n, int P, long long stride)
{
    GramGeometry g;
    g.umma = 0;
    g.NB = (n + 7) / 8;
    g.nblk = g.NB * (g.NB + 1) / 2;
    g.KG = kGramThreads / g.nblk;
    if (g.KG < 1) g.KG = 1;
    if (g.KG > 64) g.KG = 64;
    int chunks = 2;                                    // 16-byte chunks per k-row: a power of two
    while (chunks < 2 * g.NB) chunks <<= 1;
    g.NP = 4 * chunks;
    // Tile width: a whole number of columns per column group, about 16 KB of rows in flight per
    // tile, at most kPre float4 registers per thread.
    int per_group = 4096 / (g.NP * g.KG);
    if (per_group < 1) per_group = 1;
    int tk = per_group * g.KG;
    tk = (tk + 3) / 4 * 4;
    while ((long long)n * (tk / 4) > (long long)kPre * kGramThreads && tk > 4) tk -= 4;
    g.TK = tk;
    g.entries = g.nblk * 64;
    size_t tiles = sizeof(float) * 2 * (size_t)g.TK * g.NP;
    size_t scratch = sizeof(float) * 64 * kGramThreads;
    g.smem = tiles > scratch ? tiles : scratch;
    // every fp32 accumulator sums at most 4096 products before it enters fp64
    const long long max_cols = 4096LL * g.KG;
    long long cmin = (stride + max_cols - 1) / max_cols;
    const int slots = sm_count() * 2;
    long long c = (slots + P - 1) / P;
    if (c < cmin) c = cmin;
    const long long most = (stride + 127) / 128;
    if (c > most) c = most;
    if (c < 1) c = 1;
    g.cpp = (int)c;
    if (n <= 16) {   // fp32 kernel with all rows in one thread: one CTA per SM, whole waves; the running
                     // sums are flushed inside the kernel, so a CTA may take any number of tiles
        g.cpp = choose_ctas_per_partition(P, stride >> 2, kRowsTile / 4, sm_count(), 1 << 20);
    } else if (n <= 64 && stride >= kUmmaTileCols && stride < (1LL << 31) && encode_tiled_fn() != nullptr) {
        // tcgen05 kernel: 2 CTAs per SM (about 100 KB of shared memory each)
        g.umma = 1;
        // fp32 read-back sums: at most 512 flushes of 128 columns per CTA before fp64
        const long long cap_cols = 512LL * kUmmaFlushTiles * kUmmaTileCols;
        long long cmin2 = (stride + cap_cols - 1) / cap_cols;
        int c2 = choose_ctas_per_partition(P, stride >> 2, 8 * 32, sm_count() * 2);
        if (c2 < cmin2) c2 = (int)cmin2;
        g.cpp = c2;
    }
    return g;
}

int launch_gram(const GramLaunch& a, const GramGeometry& geo, cudaStream_t st)
{
    GArgs ga{a, geo};
    // shared-memory opt-in of every Gram kernel: once per device
    static std::atomic<unsigned long long> attrs_set{0};
    if (device_needs_setup(attrs_set)) {
        BTARD_CUDA_TRY(cudaFuncSetAttribute(gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
        for (int r = 4; r <= 16; r *= 2)
            for (int full = 0; full < 2; ++full)
                for (int med = 0; med < 2; ++med)
                    BTARD_CUDA_TRY(cudaFuncSetAttribute(rows_fn(r, full != 0, med != 0), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                        kRowsStages * rows_stage_bytes<16>()));
        BTARD_CUDA_TRY(cudaFuncSetAttribute(gram_umma_ws_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kWsSmem));
        BTARD_CUDA_TRY(cudaFuncSetAttribute(gram_umma_ws_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kWsSmem));
        mark_device_done(attrs_set);
    }
    if (geo.smem > 96 * 1024) return BTARD_ERR_UNSUPPORTED;
    // The tensor map of the rows is a function of (g, n, P, stride): the last one is kept per thread.
    struct MapCache { const float* g; int n, P, dev; long long stride; CUtensorMap map; bool valid; };
    static thread_local MapCache cache{};
    if (geo.umma) {
        int dev = -1;
        (void)cudaGetDevice(&dev);
        if (!(cache.valid && cache.g == a.g && cache.n == a.n && cache.P == a.P && cache.stride == a.stride && cache.dev == dev)) {
            cache.valid = false;
            if (!encode_rows_map(&cache.map, a.g, a.n, a.P, a.stride)) { set_cuda_error(cudaErrorInvalidValue); return BTARD_ERR_CUDA; }
            cache.g = a.g; cache.n = a.n; cache.P = a.P; cache.stride = a.stride; cache.dev = dev; cache.valid = true;
        }
    }
    const CUtensorMap& map = cache.map;
    prof_begin(KIND_GRAM, st);
    if (a.n <= 16) {
        const int grid = a.P * geo.cpp;
        const int R = (a.n <= 4) ? 4 : (a.n <= 8) ? 8 : 16;
        const size_t smem = (size_t)kRowsStages * (R == 4 ? rows_stage_bytes<4>() : R == 8 ? rows_stage_bytes<8>() : rows_stage_bytes<16>());
        void* args[] = {(void*)&ga};
        const cudaError_t e = cudaLaunchKernel(rows_fn(R, a.n == R, a.fuse_median != 0), dim3((unsigned)grid), dim3(kRowsThreads), args, smem, st);
        if (e != cudaSuccess) { set_cuda_error(e); prof_end(KIND_GRAM, st); return BTARD_ERR_CUDA; }
    }
    else if (geo.umma && a.n == 64) gram_umma_ws_kernel<true><<<a.P * geo.cpp, kWsThreads, kWsSmem, st>>>(ga, a.error, map);
    else if (geo.umma) gram_umma_ws_kernel<false><<<a.P * geo.cpp, kWsThreads, kWsSmem, st>>>(ga, a.error, map);
    else gram_kernel<<<a.P * geo.cpp, kGramThreads, geo.smem, st>>>(ga);
    prof_end(KIND_GRAM, st);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

int launch_gram_iterate(const GramLaunch& a, const GramGeometry& geo, cudaStream_t st)
{
    GArgs ga{a, geo};
    const size_t smem = sizeof(double) * ((size_t)a.n * a.n + a.n);
    static std::atomic<unsigned long long> attrs_set{0};
    if (device_needs_setup(attrs_set)) {      // n <= 128: at most 129 KB
        BTARD_CUDA_TRY(cudaFuncSetAttribute(gram_iterate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 132 * 1024));
        mark_device_done(attrs_set);
    }
    prof_begin(KIND_COEF, st);
    if (a.n <= 16) gram_iterate_warp_kernel<16><<<a.P, 32, 0, st>>>(ga);
    else if (a.n <= 32) gram_iterate_warp_kernel<32><<<a.P, 32, 0, st>>>(ga);
    else gram_iterate_kernel<<<a.P, kGramThreads, smem, st>>>(ga);
    prof_end(KIND_COEF, st);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

int launch_gram_finalize(const double* tot, double* resid_norm, uint32_t* status, int n, int P,
                         const unsigned int* error, cudaStream_t st)
{
    gram_finalize_kernel<<<P, 128, 0, st>>>(tot, resid_norm, status, n, error);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

}  // namespace btard
