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
// G is a dense contraction over the columns.  It is computed here on the fp32 FMA pipes: the
// products of residuals that differ by orders of magnitude (attacked rows) must stay accurate to
// about 1e-6 relative for the subtraction above, which rules out single-pass TF32.
#include "btard_common.h"

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
                    const float4 x = __ldcs(reinterpret_cast<const float4*>(gp + (size_t)row * stride + col));
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

// ---- n <= 16: the Gram block on the tensor cores, straight from registers ------------------------
// One warp owns 16 rows x 16 columns at a time.  In the m16n8k8 fragment layout the B operand of
// R R^T is the A operand itself (lane (g, t) holds rows g, g+8 and the same four columns for both),
// so nothing is staged in shared memory.  TF32 alone would lose the low 13 bits of every residual;
// each value is split as hi + lo (both TF32) and hi.hi + hi.lo + lo.hi is accumulated, which keeps
// products to about 2^-21.  The tensor core adds with truncation, so its accumulator only ever
// holds one 16-column block (6 chained MMAs); blocks are summed on the fp32 pipe (round to
// nearest) and moved to fp64 every 64 blocks.
__device__ __forceinline__ uint32_t to_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

constexpr int kMmaStepCols = 64;      // columns a warp takes per step (4 blocks of 16)

__global__ void __launch_bounds__(kGramThreads) gram_mma16_kernel(const GArgs k)
{
    __shared__ double sh_tile[kGramThreads / 32][16][16];
    __shared__ int sh_last;
    const GramLaunch& a = k.a;
    const int n = a.n, cpp = k.g.cpp, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const long long stride = a.stride, len = a.table[p].len;
    const float* gp = a.g + (size_t)p * n * stride;
    const float* vp = a.v0 + (size_t)p * stride;
    long long c0 = stride * j / cpp, c1 = stride * (j + 1) / cpp;
    if (j > 0) c0 &= ~31LL;
    if (j + 1 < cpp) c1 &= ~31LL;

    const bool row0 = g < n, row1 = g + 8 < n;
    const float* p0 = gp + (size_t)g * stride;
    const float* p1 = gp + (size_t)(g + 8) * stride;

    float sum0[4] = {0.f, 0.f, 0.f, 0.f}, sum1[4] = {0.f, 0.f, 0.f, 0.f};     // fp32 running sums
    double big0[4] = {0., 0., 0., 0.}, big1[4] = {0., 0., 0., 0.};
    int since_flush = 0;

    for (long long cs = c0 + (long long)warp * kMmaStepCols; cs < c1; cs += (long long)(kGramThreads / 32) * kMmaStepCols) {
        float4 x0[4], x1[4], v4[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {                  // all loads of the step first
            const long long col = cs + 16 * b + 4 * t;
            const bool in = col < c1;
            x0[b] = (in && row0) ? __ldcs(reinterpret_cast<const float4*>(p0 + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            x1[b] = (in && row1) ? __ldcs(reinterpret_cast<const float4*>(p1 + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            v4[b] = in ? *reinterpret_cast<const float4*>(vp + col) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const long long col = cs + 16 * b + 4 * t;
            const bool m0 = col < len && col < c1, m1 = col + 1 < len && col < c1;
            const bool m2 = col + 2 < len && col < c1, m3 = col + 3 < len && col < c1;
            // residuals of rows g and g+8 at this lane's four columns
            const float r0[4] = {(m0 && row0) ? x0[b].x - v4[b].x : 0.f, (m1 && row0) ? x0[b].y - v4[b].y : 0.f,
                                 (m2 && row0) ? x0[b].z - v4[b].z : 0.f, (m3 && row0) ? x0[b].w - v4[b].w : 0.f};
            const float r1[4] = {(m0 && row1) ? x1[b].x - v4[b].x : 0.f, (m1 && row1) ? x1[b].y - v4[b].y : 0.f,
                                 (m2 && row1) ? x1[b].z - v4[b].z : 0.f, (m3 && row1) ? x1[b].w - v4[b].w : 0.f};
            uint32_t h0[4], h1[4], l0[4], l1[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                h0[q] = to_tf32(r0[q]);
                h1[q] = to_tf32(r1[q]);
                l0[q] = to_tf32(r0[q] - __uint_as_float(h0[q]));
                l1[q] = to_tf32(r1[q] - __uint_as_float(h1[q]));
            }
            float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {           // two k-steps: columns (0,1) then (2,3) of the lane
                const int qa = 2 * ks, qb = 2 * ks + 1;
                const uint32_t ah[4] = {h0[qa], h1[qa], h0[qb], h1[qb]};
                const uint32_t al[4] = {l0[qa], l1[qa], l0[qb], l1[qb]};
                // columns 0..7 of G: B = rows g of R; columns 8..15: rows g+8
                mma_tf32(d0, ah, h0[qa], h0[qb]);
                mma_tf32(d0, ah, l0[qa], l0[qb]);
                mma_tf32(d0, al, h0[qa], h0[qb]);
                mma_tf32(d1, ah, h1[qa], h1[qb]);
                mma_tf32(d1, ah, l1[qa], l1[qb]);
                mma_tf32(d1, al, h1[qa], h1[qb]);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) { sum0[q] += d0[q]; sum1[q] += d1[q]; }
        }
        if (++since_flush == 16) {                     // 64 blocks of 16 columns
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                big0[q] += (double)sum0[q]; big1[q] += (double)sum1[q];
                sum0[q] = 0.f; sum1[q] = 0.f;
            }
            since_flush = 0;
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) { big0[q] += (double)sum0[q]; big1[q] += (double)sum1[q]; }

    // accumulator fragment: (row g, col 2t), (g, 2t+1), (g+8, 2t), (g+8, 2t+1); d1 is 8 columns on
    sh_tile[warp][g][2 * t] = big0[0];
    sh_tile[warp][g][2 * t + 1] = big0[1];
    sh_tile[warp][g + 8][2 * t] = big0[2];
    sh_tile[warp][g + 8][2 * t + 1] = big0[3];
    sh_tile[warp][g][8 + 2 * t] = big1[0];
    sh_tile[warp][g][8 + 2 * t + 1] = big1[1];
    sh_tile[warp][g + 8][8 + 2 * t] = big1[2];
    sh_tile[warp][g + 8][8 + 2 * t + 1] = big1[3];
    __syncthreads();
    const int entries = k.g.entries, NB = k.g.NB;
    double* slots = a.slots + (size_t)p * cpp * entries;
    double* dst = slots + (size_t)j * entries;
    for (int idx = tid; idx < entries; idx += kGramThreads) {
        const int b = idx >> 6, e = idx & 63;
        int bi, bj;
        block_coords(b, NB, bi, bj);
        const int r = 8 * bi + (e >> 3), c = 8 * bj + (e & 7);
        double s = 0.0;
        for (int w = 0; w < kGramThreads / 32; ++w) s += sh_tile[w][r][c];
        dst[idx] = s;
    }
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

// ---- 17 <= n <= 64: the Gram block on the 5th-generation tensor cores (tcgen05 + TMEM) ----------
// Per 32-column tile the CTA's threads form R = g - v0, split every value into TF32 hi + lo and write
// both as K-major operand tiles (128-byte rows, 128-byte swizzle) into shared memory; one thread then
// issues, per 8-column k-block, three tcgen05.mma (hi.hi, hi.lo, lo.hi) with M = 64 (rows n..63 are
// zero), N = 64, accumulating G in 64 columns of tensor memory (row m of G lives in lane
// m % 16 + 32 (m / 16): sixteen rows in the lower half of each warp's quarter).  A and B descriptors point at the
// same tiles: B = R.  Two stages alternate, an mbarrier per stage (armed by tcgen05.commit) tells when
// the tensor core has finished reading it.  Because tensor-core accumulation truncates, the
// accumulator is read back (tcgen05.ld) and restarted every 4 tiles; the read-back values are summed
// on the fp32 pipe and turned into fp64 at the end.  Every wait is bounded; if one expires the CTA
// raises the error flag, still frees its tensor memory and leaves.
constexpr int kUmmaThreads = 128;
constexpr int kUmmaTileCols = 32;                       // one 128-byte swizzle row of TF32
constexpr int kUmmaTileBytes = 64 * 128;                // 64 rows x 128 bytes
constexpr int kUmmaFlushTiles = 4;
constexpr int kUmmaSpinLimit = 1 << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    // K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; descriptor version 1 (sm_100)
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (int spin = 0; spin < kUmmaSpinLimit; ++spin) {
        uint32_t done;
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.b32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
        __nanosleep(32);                               // do not burn issue slots while the tensor core works
    }
    return false;
}

__global__ void __launch_bounds__(kUmmaThreads) gram_umma_kernel(const GArgs k, unsigned int* error)
{
    extern __shared__ __align__(1024) unsigned char sh_raw[];
    __shared__ __align__(8) unsigned long long sh_mbar[2];
    __shared__ uint32_t sh_tmem;
    __shared__ int sh_last;
    const GramLaunch& a = k.a;
    const int n = a.n, cpp = k.g.cpp, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int p = blockIdx.x / cpp, j = blockIdx.x % cpp;
    const long long stride = a.stride, len = a.table[p].len;
    const float* gp = a.g + (size_t)p * n * stride;
    const float* vp = a.v0 + (size_t)p * stride;
    // The CTAs of a partition take its 32-column tiles round-robin (tile j, j + cpp, ...): they are
    // resident together, so at any moment they read neighbouring 128-byte pieces of the same rows and
    // an open DRAM page is used whole instead of 128 bytes at a time.
    const long long c1 = stride;
    const long long all_tiles = (stride + kUmmaTileCols - 1) / kUmmaTileCols;
    const int ntiles = (int)((all_tiles - j + cpp - 1) / cpp);      // tiles j + m cpp < all_tiles
    auto tile_col = [&](int t) { return ((long long)j + (long long)t * cpp) * kUmmaTileCols; };

    // operand tiles: [stage][hi, lo][64 rows][128 bytes], 1024-byte aligned
    unsigned char* tiles = (unsigned char*)(((uintptr_t)sh_raw + 1023) & ~(uintptr_t)1023);
    for (int e = tid; e < 4 * kUmmaTileBytes / 16; e += kUmmaThreads)
        reinterpret_cast<uint4*>(tiles)[e] = make_uint4(0u, 0u, 0u, 0u);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_mbar[0])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh_mbar[1])));
    }
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh_tmem)), "r"(64));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sh_tmem;

    // tf32 inputs, fp32 accumulate, K-major A and B, N = 64, M = 64
    const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((64u >> 3) << 17) | ((64u >> 4) << 24);
    const uint32_t tile_base = smem_u32(tiles);

    float sum[64];
#pragma unroll
    for (int q = 0; q < 64; ++q) sum[q] = 0.0f;
    int commits[2] = {0, 0};
    bool failed = false;
    int since_flush = 0;
    __shared__ int sh_fail;
    if (tid == 0) sh_fail = 0;

    // this thread's four 16-byte chunks of a tile: rows row0 + 16 i, chunk ch (4 columns);
    // the rows of the next two tiles are kept in flight in registers
    const int row0 = tid >> 3, ch = tid & 7;
    float4 xa[4], xb[4], va, vb;
    auto fetch = [&](int t, float4 (&x)[4], float4& v4) {
        const long long col = tile_col(t) + 4 * ch;
        const bool in = t < ntiles && col < c1;
        v4 = in ? *reinterpret_cast<const float4*>(vp + col) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = row0 + 16 * i;
            x[i] = (in && r < n) ? __ldcs(reinterpret_cast<const float4*>(gp + (size_t)r * stride + col))
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    // 32 accumulator columns starting at column `first` of this warp's 32 lanes, added to sum
    auto read_back = [&](uint32_t taddr, float* dst) {
        uint32_t d[32];
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
            "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
            : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]),
              "=r"(d[8]), "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15]),
              "=r"(d[16]), "=r"(d[17]), "=r"(d[18]), "=r"(d[19]), "=r"(d[20]), "=r"(d[21]), "=r"(d[22]), "=r"(d[23]),
              "=r"(d[24]), "=r"(d[25]), "=r"(d[26]), "=r"(d[27]), "=r"(d[28]), "=r"(d[29]), "=r"(d[30]), "=r"(d[31])
            : "r"(taddr));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int q = 0; q < 32; ++q) dst[q] += __uint_as_float(d[q]);
    };

    fetch(0, xa, va);
    fetch(1, xb, vb);
    __syncthreads();
    for (int t = 0; t < ntiles; ++t) {
        const int s = t & 1;
        // the tensor core must be done with what it read from this stage two tiles ago
        if (commits[s] > 0 && !mbar_wait(smem_u32(&sh_mbar[s]), (uint32_t)((commits[s] - 1) & 1))) sh_fail = 1;

        const long long col = tile_col(t) + 4 * ch;
        const bool m0 = col < len && col < c1, m1 = col + 1 < len && col < c1;
        const bool m2 = col + 2 < len && col < c1, m3 = col + 3 < len && col < c1;
        unsigned char* hi_tile = tiles + (size_t)(2 * s) * kUmmaTileBytes;
        unsigned char* lo_tile = hi_tile + kUmmaTileBytes;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = row0 + 16 * i;
            if (r < n) {
                const float r0 = m0 ? xa[i].x - va.x : 0.f, r1 = m1 ? xa[i].y - va.y : 0.f;
                const float r2 = m2 ? xa[i].z - va.z : 0.f, r3 = m3 ? xa[i].w - va.w : 0.f;
                const uint32_t h0 = to_tf32(r0), h1 = to_tf32(r1), h2 = to_tf32(r2), h3 = to_tf32(r3);
                const uint32_t l0 = to_tf32(r0 - __uint_as_float(h0)), l1 = to_tf32(r1 - __uint_as_float(h1));
                const uint32_t l2 = to_tf32(r2 - __uint_as_float(h2)), l3 = to_tf32(r3 - __uint_as_float(h3));
                const int off = (r >> 3) * 1024 + (r & 7) * 128 + ((ch ^ (r & 7)) << 4);
                *reinterpret_cast<uint4*>(hi_tile + off) = make_uint4(h0, h1, h2, h3);
                *reinterpret_cast<uint4*>(lo_tile + off) = make_uint4(l0, l1, l2, l3);
            }
        }
        // rotate the register queue and put tile t + 2 in flight
#pragma unroll
        for (int i = 0; i < 4; ++i) xa[i] = xb[i];
        va = vb;
        fetch(t + 2, xb, vb);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (sh_fail) { failed = true; break; }         // a bounded wait ran out somewhere in the CTA
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t hi_addr = tile_base + (uint32_t)(2 * s) * kUmmaTileBytes;
            const uint32_t lo_addr = hi_addr + kUmmaTileBytes;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {           // 8 TF32 = 32 bytes per k-block
                const uint64_t dh = umma_desc(hi_addr + 32u * ks), dl = umma_desc(lo_addr + 32u * ks);
                const uint32_t acc0 = (since_flush > 0 || ks > 0) ? 1u : 0u;
                asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
                             ::"r"(tmem), "l"(dh), "l"(dh), "r"(idesc), "r"(acc0) : "memory");
                asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
                             ::"r"(tmem), "l"(dh), "l"(dl), "r"(idesc), "r"(1u) : "memory");
                asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
                             ::"r"(tmem), "l"(dl), "l"(dh), "r"(idesc), "r"(1u) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                         ::"r"(smem_u32(&sh_mbar[s])) : "memory");
        }
        commits[s] += 1;
        since_flush += 1;

        if (since_flush == kUmmaFlushTiles || t + 1 == ntiles) {
            // read the accumulator back: wait for the commit just issued (covers all earlier MMAs)
            if (!mbar_wait(smem_u32(&sh_mbar[s]), (uint32_t)((commits[s] - 1) & 1))) sh_fail = 1;
            __syncthreads();
            if (sh_fail) { failed = true; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            {                                          // lanes 0..15 of every warp: rows 16 warp + lane
                const uint32_t taddr = tmem + ((uint32_t)(32 * warp) << 16);
                read_back(taddr, sum);
                read_back(taddr + 32u, sum + 32);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncthreads();
            since_flush = 0;
        }
    }
    if (failed && tid == 0) atomicExch(error, 1u);

    // leave tensor memory the way it was found
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(64));
    }

    // row i = 16 warp + lane of G (lanes 0..15) -> fp64 matrix in shared memory -> this CTA's slot
    double* sh_g = reinterpret_cast<double*>(tiles);     // [64][64], the operand tiles are dead now
    __syncthreads();
    if (lane < 16) {
        const int i = 16 * warp + lane;
#pragma unroll
        for (int q = 0; q < 64; ++q) sh_g[i * 64 + q] = (double)sum[q];
    }
    __syncthreads();
    const int entries = k.g.entries, NB = k.g.NB;
    double* slots = a.slots + (size_t)p * cpp * entries;
    double* dst = slots + (size_t)j * entries;
    for (int idx = tid; idx < entries; idx += kUmmaThreads) {
        const int b = idx >> 6, e = idx & 63;
        int bi, bj;
        block_coords(b, NB, bi, bj);
        dst[idx] = sh_g[(8 * bi + (e >> 3)) * 64 + 8 * bj + (e & 7)];
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) sh_last = (atomicAdd(&a.ticket[p], 1u) == (unsigned)(cpp - 1));
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    double* out = a.gram + (size_t)p * entries;
    for (int idx = tid; idx < entries; idx += kUmmaThreads) {
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
        double w = 0.0;
        if (row && !bad) {
            double rho2 = gii - 2.0 * Gai + aGa;
            if (rho2 < 0.0) rho2 = 0.0;
            const double rho = sqrt(rho2);
            if (isfinite(rho)) w = (rho <= tau) ? 1.0 : tau / rho;
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
__device__ __forceinline__ double warp_allsum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <int N>   // 16 or 32: rows of G held per lane
__global__ void __launch_bounds__(32) gram_iterate_warp_kernel(const GArgs k)
{
    const GramLaunch& a = k.a;
    const int n = a.n, NB = k.g.NB, lane = threadIdx.x, p = blockIdx.x;
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
    double ai = 0.0, Gai = 0.0, step2 = 0.0;
    int iters = 0;
    for (int l = 0; l < a.max_iters; ++l) {
        const double aGa = warp_allsum(live ? ai * Gai : 0.0);
        double w = 0.0;
        if (live) {
            double rho2 = gii - 2.0 * Gai + aGa;
            if (rho2 < 0.0) rho2 = 0.0;
            const double rho = sqrt(rho2);
            if (isfinite(rho)) w = (rho <= tau) ? 1.0 : tau / rho;
        }
        const double W = warp_allsum(w);
        const double d = live ? (w - W * ai) / (double)n : 0.0;
        double Gd = 0.0;
#pragma unroll
        for (int q = 0; q < N; ++q) {
            const double dq = __shfl_sync(0xffffffffu, d, q);
            if (dq != 0.0 && live) Gd += Grow[q] * dq;
        }
        step2 = warp_allsum(live ? d * Gd : 0.0);
        ai += d;
        Gai += Gd;
        iters = l + 1;
        if (a.stop_mode == BTARD_STOP_EPS && step2 <= a.eps2) break;
    }
    if (step2 < 0.0) step2 = 0.0;
    if (row) a.coef[(size_t)p * n + lane] = ai;
    const unsigned anybad = __ballot_sync(0xffffffffu, bad);
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

}  // namespace

GramGeometry gram_geometry(int n, int P, long long stride)
{
    GramGeometry g;
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
    if (n <= 16) {   // tensor-core kernel: whole waves of resident CTAs
        int nb = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, gram_mma16_kernel, kGramThreads, 0) != cudaSuccess || nb < 1) {
            (void)cudaGetLastError();
            nb = 2;
        }
        g.cpp = choose_ctas_per_partition(P, stride >> 2, 16 * (kGramThreads / 32), sm_count() * nb);
    } else if (n <= 64) {   // tcgen05 kernel: 3 CTAs per SM (160 registers x 128 threads each)
        // fp32 read-back sums: at most 512 flushes of 128 columns per CTA before fp64
        const long long cap_cols = 512LL * kUmmaFlushTiles * kUmmaTileCols;
        long long cmin2 = (stride + cap_cols - 1) / cap_cols;
        int c2 = choose_ctas_per_partition(P, stride >> 2, 8 * 32, sm_count() * 3);
        if (c2 < cmin2) c2 = (int)cmin2;
        g.cpp = c2;
    }
    return g;
}

int launch_gram(const GramLaunch& a, const GramGeometry& geo, cudaStream_t st)
{
    GArgs ga{a, geo};
    if (geo.smem > 48 * 1024)
        BTARD_CUDA_TRY(cudaFuncSetAttribute(gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)geo.smem));
    constexpr int umma_smem = 4 * kUmmaTileBytes + 1024;
    if (a.n > 16 && a.n <= 64)
        BTARD_CUDA_TRY(cudaFuncSetAttribute(gram_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, umma_smem));
    prof_begin(KIND_GRAM, st);
    if (a.n <= 16) gram_mma16_kernel<<<a.P * geo.cpp, kGramThreads, 0, st>>>(ga);
    else if (a.n <= 64) gram_umma_kernel<<<a.P * geo.cpp, kUmmaThreads, umma_smem, st>>>(ga, a.error);
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
    if (smem > 48 * 1024)
        BTARD_CUDA_TRY(cudaFuncSetAttribute(gram_iterate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
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
