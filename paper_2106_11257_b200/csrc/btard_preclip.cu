// Per-part gradient clipping of BTARD-Clipped-SGD (Alg. 9 and the paragraph after it):
//     g~_i(l) = min{1, lambda / ||g_i(l)||_2} g_i(l)     for every peer i and part l,
// applied in place to the [P][n][row_stride] tensor before it is aggregated.  Two streaming kernels:
// squared row norms (per-chunk partial sums in slots, no atomics), then every chunk adds up its row's
// slots in a fixed order and rescales its piece of the row, writing only rows that are actually clipped.
#include "btard_common.h"

namespace btard {
namespace {

constexpr int kPreThreads = 256;

__device__ __forceinline__ double block_sum_256(double x, double* red)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    double s = 0.0;
    for (int w = 0; w < kPreThreads / 32; ++w) s += red[w];
    return s;
}

struct PreArgs {
    float* g;
    const PartEntry* table;     // len, and lambda in the tau field
    double* slots;              // [P*n][chunks]
    double* row_norm;           // [P][n] out
    double* factor;             // [P][n] out
    uint32_t* status;           // [P] out
    long long stride;
    int n, P, chunks;
    int rewrite;                // 1: rescale the clipped rows in place; -1: norms and factors only (one CTA per row)
};

__device__ __forceinline__ void chunk_range(long long quads, int c, int chunks, long long& q0, long long& q1)
{
    q0 = quads * c / chunks;
    q1 = quads * (c + 1) / chunks;
    if (c > 0) q0 &= ~7LL;
    if (c + 1 < chunks) q1 &= ~7LL;
}

__global__ void __launch_bounds__(kPreThreads) preclip_norm_kernel(const PreArgs a)
{
    __shared__ double red[kPreThreads / 32];
    const long long row = blockIdx.x / a.chunks;
    const int c = blockIdx.x % a.chunks, p = (int)(row / a.n);
    const long long len = a.table[p].len;
    const float* x = a.g + (size_t)row * a.stride;
    long long q0, q1;
    chunk_range(a.stride >> 2, c, a.chunks, q0, q1);
    double acc = 0.0;
    float part = 0.0f;
    int run = 0;
    for (long long q = q0 + threadIdx.x; q < q1; q += kPreThreads) {
        const long long col = 4 * q;
        if (col >= len) break;
        const float4 v = __ldg(reinterpret_cast<const float4*>(x + col));
        part += v.x * v.x;
        if (col + 1 < len) part += v.y * v.y;
        if (col + 2 < len) part += v.z * v.z;
        if (col + 3 < len) part += v.w * v.w;
        if (++run == 64) { acc += (double)part; part = 0.0f; run = 0; }   // short fp32 runs only
    }
    acc += (double)part;
    const double s = block_sum_256(acc, red);
    if (threadIdx.x == 0) a.slots[(size_t)row * a.chunks + c] = s;
}

__global__ void __launch_bounds__(kPreThreads) preclip_scale_kernel(const PreArgs a)
{
    __shared__ double sh_norm2;
    // rewrite < 0: one CTA per row, norms and factors only
    const long long row = (a.rewrite < 0) ? blockIdx.x : blockIdx.x / a.chunks;
    const int c = (a.rewrite < 0) ? 0 : blockIdx.x % a.chunks, p = (int)(row / a.n);
    const long long len = a.table[p].len;
    const double lambda = a.table[p].tau;
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int q = 0; q < a.chunks; ++q) s += a.slots[(size_t)row * a.chunks + q];
        sh_norm2 = s;
    }
    __syncthreads();
    const double norm = sqrt(sh_norm2);
    double f;
    if (!isfinite(norm)) f = 0.0;                     // a non-finite row is dropped (set to zero)
    else f = (norm <= lambda) ? 1.0 : lambda / norm;
    if (c == 0 && threadIdx.x == 0) {
        a.row_norm[row] = norm;
        a.factor[row] = f;
        if (!isfinite(norm)) atomicOr(&a.status[p], BTARD_STATUS_NONFINITE_ROW);
    }
    if (f == 1.0 || a.rewrite <= 0) return;               // untouched rows cost no write traffic
    float* x = a.g + (size_t)row * a.stride;
    long long q0, q1;
    chunk_range(a.stride >> 2, c, a.chunks, q0, q1);
    const float ff = (float)f;
    for (long long q = q0 + threadIdx.x; q < q1; q += kPreThreads) {
        const long long col = 4 * q;
        if (col >= len) break;
        float4 v = *reinterpret_cast<const float4*>(x + col);
        if (f == 0.0) v = make_float4(0.f, 0.f, 0.f, 0.f);
        else { v.x *= ff; v.y *= ff; v.z *= ff; v.w *= ff; }
        *reinterpret_cast<float4*>(x + col) = v;      // columns past len are padding: any value is fine
    }
}

__global__ void preclip_reset_kernel(uint32_t* status, int P)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p < P) status[p] = 0;
}

}  // namespace

int preclip_chunks(int n, int P, long long stride)
{
    const long long rows = (long long)n * P;
    long long want = (4LL * sm_count() * 4 + rows - 1) / rows;      // about four waves of 4 CTAs per SM
    const long long most = ((stride >> 2) + 2047) / 2048;           // at least 32 KB of a row per CTA
    if (want > most) want = most;
    if (want < 1) want = 1;
    return (int)want;
}

int launch_preclip(float* g, const PartEntry* table, double* slots, double* row_norm, double* factor,
                   uint32_t* status, long long stride, int n, int P, int chunks, bool rewrite, cudaStream_t st)
{
    PreArgs a{g, table, slots, row_norm, factor, status, stride, n, P, chunks, rewrite ? 1 : 0};
    const long long grid = (long long)n * P * chunks;
    if (grid > 0x7fffffffLL) return BTARD_ERR_UNSUPPORTED;
    preclip_reset_kernel<<<(P + 127) / 128, 128, 0, st>>>(status, P);
    preclip_norm_kernel<<<(unsigned)grid, kPreThreads, 0, st>>>(a);
    // without the rewrite one CTA per row is enough: it adds up the slots and writes norm and factor
    if (rewrite) preclip_scale_kernel<<<(unsigned)grid, kPreThreads, 0, st>>>(a);
    else preclip_scale_kernel<<<(unsigned)((long long)n * P), 32, 0, st>>>(PreArgs{g, table, slots, row_norm, factor, status, stride, n, P, chunks, -1});
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch(3);
    return BTARD_OK;
}

}  // namespace btard
