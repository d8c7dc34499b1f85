// Split and Merge of App. D.1 as device copies: the n gradient vectors [n][d] become the slab tensor
// [P][n][row_stride] that the aggregation reads (this is what the all-to-all of Alg. 2 (every peer sends part j to aggregator j)
// delivers when every peer is a row of one GPU), and the aggregated parts [P][row_stride] are
// concatenated back into one vector of d coordinates (Alg. 2, Merge).  Source offsets are arbitrary,
// so the copies use coalesced 32-bit accesses; padding columns are written as zero.
#include "btard_common.h"

namespace btard {
namespace {

struct PackEntry { long long offset, len; };

__global__ void __launch_bounds__(256) split_kernel(const float* grads, float* g, const PackEntry* tab,
                                                    long long d, long long stride, int n)
{
    const long long row = blockIdx.y;                  // p * n + i
    const int p = (int)(row / n), i = (int)(row % n);
    const long long off = tab[p].offset, len = tab[p].len;
    const float* src = grads + (size_t)i * d + off;
    float* dst = g + (size_t)row * stride;
    for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < stride;
         c += (long long)gridDim.x * blockDim.x)
        dst[c] = (c < len) ? __ldg(src + c) : 0.0f;
}

__global__ void __launch_bounds__(256) merge_kernel(const float* v, float* out, const PackEntry* tab,
                                                    long long stride)
{
    const int p = blockIdx.y;
    const long long off = tab[p].offset, len = tab[p].len;
    const float* src = v + (size_t)p * stride;
    for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < len;
         c += (long long)gridDim.x * blockDim.x)
        out[off + c] = src[c];
}

}  // namespace

int launch_split(const float* grads, float* g, const void* table_dev, long long d, long long stride,
                 int n, int P, cudaStream_t st)
{
    const long long rows = (long long)n * P;
    if (rows > 65535) return BTARD_ERR_UNSUPPORTED;
    long long bx = (stride + 256 * 8 - 1) / (256 * 8);
    if (bx < 1) bx = 1;
    if (bx > 4096) bx = 4096;
    split_kernel<<<dim3((unsigned)bx, (unsigned)rows), 256, 0, st>>>(grads, g, (const PackEntry*)table_dev, d, stride, n);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

int launch_merge(const float* v, float* out, const void* table_dev, long long stride, int P, cudaStream_t st)
{
    long long bx = (stride + 256 * 8 - 1) / (256 * 8);
    if (bx < 1) bx = 1;
    if (bx > 4096) bx = 4096;
    merge_kernel<<<dim3((unsigned)bx, (unsigned)P), 256, 0, st>>>(v, out, (const PackEntry*)table_dev, stride);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch();
    return BTARD_OK;
}

}  // namespace btard
