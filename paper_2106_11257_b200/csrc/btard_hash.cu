// Commitments of Alg. 2 (lines 2 and 6: peers broadcast hash(g_i[j]) and hash(g^_i) before the parts
// travel).  The paper only asks for a cryptographic hash; this build fixes SHA-256 (FIPS 180-4) in a
// two-level tree so that a multi-megabyte part is hashed by thousands of threads:
//     H(row) = SHA256( SHA256(chunk_0) || SHA256(chunk_1) || ... || LE64(byte length) ),
// chunks = consecutive 4096-byte pieces of the row's 4 * part_len bytes (the last one may be shorter;
// an empty row has none).  Bytes are the float32 values as they lie in memory (little endian).
// Integer work only; results are bit-exact.
#include "btard_common.h"

namespace btard {
namespace {

constexpr int kLeafBytes = 4096;

__constant__ uint32_t kSha[64] = {
    0x428a2f98u, 0x71374491u, 0xb5c0fbcfu, 0xe9b5dba5u, 0x3956c25bu, 0x59f111f1u, 0x923f82a4u, 0xab1c5ed5u,
    0xd807aa98u, 0x12835b01u, 0x243185beu, 0x550c7dc3u, 0x72be5d74u, 0x80deb1feu, 0x9bdc06a7u, 0xc19bf174u,
    0xe49b69c1u, 0xefbe4786u, 0x0fc19dc6u, 0x240ca1ccu, 0x2de92c6fu, 0x4a7484aau, 0x5cb0a9dcu, 0x76f988dau,
    0x983e5152u, 0xa831c66du, 0xb00327c8u, 0xbf597fc7u, 0xc6e00bf3u, 0xd5a79147u, 0x06ca6351u, 0x14292967u,
    0x27b70a85u, 0x2e1b2138u, 0x4d2c6dfcu, 0x53380d13u, 0x650a7354u, 0x766a0abbu, 0x81c2c92eu, 0x92722c85u,
    0xa2bfe8a1u, 0xa81a664bu, 0xc24b8b70u, 0xc76c51a3u, 0xd192e819u, 0xd6990624u, 0xf40e3585u, 0x106aa070u,
    0x19a4c116u, 0x1e376c08u, 0x2748774cu, 0x34b0bcb5u, 0x391c0cb3u, 0x4ed8aa4au, 0x5b9cca4fu, 0x682e6ff3u,
    0x748f82eeu, 0x78a5636fu, 0x84c87814u, 0x8cc70208u, 0x90befffau, 0xa4506cebu, 0xbef9a3f7u, 0xc67178f2u};

__device__ __forceinline__ uint32_t rotr(uint32_t x, int n) { return __funnelshift_r(x, x, n); }

struct Sha {
    uint32_t h[8];
    __device__ void init()
    {
        h[0] = 0x6a09e667u; h[1] = 0xbb67ae85u; h[2] = 0x3c6ef372u; h[3] = 0xa54ff53au;
        h[4] = 0x510e527fu; h[5] = 0x9b05688cu; h[6] = 0x1f83d9abu; h[7] = 0x5be0cd19u;
    }
    // one 64-byte block given as 16 big-endian words
    __device__ void block(uint32_t (&w)[16])
    {
        uint32_t a = h[0], b = h[1], c = h[2], d = h[3], e = h[4], f = h[5], g = h[6], hh = h[7];
#pragma unroll
        for (int i = 0; i < 64; ++i) {
            if (i >= 16) {
                const uint32_t w15 = w[(i + 1) & 15], w2 = w[(i + 14) & 15];
                const uint32_t s0 = rotr(w15, 7) ^ rotr(w15, 18) ^ (w15 >> 3);
                const uint32_t s1 = rotr(w2, 17) ^ rotr(w2, 19) ^ (w2 >> 10);
                w[i & 15] = w[i & 15] + s0 + w[(i + 9) & 15] + s1;
            }
            const uint32_t t1 = hh + (rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25)) + ((e & f) ^ (~e & g)) + kSha[i] + w[i & 15];
            const uint32_t t2 = (rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22)) + ((a & b) ^ (a & c) ^ (b & c));
            hh = g; g = f; f = e; e = d + t1; d = c; c = b; b = a; a = t1 + t2;
        }
        h[0] += a; h[1] += b; h[2] += c; h[3] += d; h[4] += e; h[5] += f; h[6] += g; h[7] += hh;
    }
};

// SHA-256 of `bytes` bytes (a multiple of 4) starting at the 4-byte aligned `src`; 32-bit little-endian
// memory words are byte-swapped into the big-endian words the standard works on.
__device__ void sha256_words(const uint32_t* src, long long bytes, uint32_t (&digest)[8])
{
    Sha s;
    s.init();
    const long long nwords = bytes >> 2;
    long long at = 0;
    uint32_t w[16];
    for (; at + 16 <= nwords; at += 16) {
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = __byte_perm(src[at + i], 0, 0x0123);
        s.block(w);
    }
    const int rest = (int)(nwords - at);               // 0..15 words left, then the padding
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = (i < rest) ? __byte_perm(src[at + i], 0, 0x0123) : 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i)
        if (i == rest) w[i] = 0x80000000u;
    if (rest >= 14) {                                  // no room for the length: one more block
        s.block(w);
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = 0u;
    }
    const unsigned long long bits = (unsigned long long)bytes * 8ull;
    w[14] = (uint32_t)(bits >> 32);
    w[15] = (uint32_t)bits;
    s.block(w);
#pragma unroll
    for (int i = 0; i < 8; ++i) digest[i] = s.h[i];
}

struct HashArgs {
    const float* x;             // [rows][stride]
    const PartEntry* table;     // len per partition (rows_per_part rows each)
    uint32_t* leaves;           // [rows][max_leaves][8] big-endian digest words
    unsigned char* out;         // [rows][32]
    long long stride;
    int rows_per_part, rows, max_leaves;
};

__global__ void __launch_bounds__(128) hash_leaves_kernel(const HashArgs a)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long row = t / a.max_leaves;
    const int leaf = (int)(t % a.max_leaves);
    if (row >= a.rows) return;
    const long long bytes = 4 * a.table[row / a.rows_per_part].len;
    const long long start = (long long)leaf * kLeafBytes;
    if (start >= bytes) return;
    const long long nb = (bytes - start < kLeafBytes) ? bytes - start : kLeafBytes;
    uint32_t dg[8];
    sha256_words(reinterpret_cast<const uint32_t*>(a.x + (size_t)row * a.stride) + (start >> 2), nb, dg);
    uint32_t* dst = a.leaves + ((size_t)row * a.max_leaves + leaf) * 8;
#pragma unroll
    for (int i = 0; i < 8; ++i) dst[i] = __byte_perm(dg[i], 0, 0x0123);   // stored as digest bytes
}

__global__ void __launch_bounds__(128) hash_roots_kernel(const HashArgs a)
{
    const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= a.rows) return;
    const long long bytes = 4 * a.table[row / a.rows_per_part].len;
    const long long nleaves = (bytes + kLeafBytes - 1) / kLeafBytes;
    // message: nleaves digests (32 bytes each) followed by the byte length as 8 little-endian bytes
    uint32_t* msg = a.leaves + (size_t)row * a.max_leaves * 8;
    // the length is appended in place behind the digests (room is reserved: max_leaves counts it)
    msg[nleaves * 8] = (uint32_t)((unsigned long long)bytes & 0xffffffffull);
    msg[nleaves * 8 + 1] = (uint32_t)((unsigned long long)bytes >> 32);
    uint32_t dg[8];
    sha256_words(msg, nleaves * 32 + 8, dg);
    unsigned char* o = a.out + (size_t)row * 32;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        o[4 * i] = (unsigned char)(dg[i] >> 24);
        o[4 * i + 1] = (unsigned char)(dg[i] >> 16);
        o[4 * i + 2] = (unsigned char)(dg[i] >> 8);
        o[4 * i + 3] = (unsigned char)dg[i];
    }
}

}  // namespace

int hash_max_leaves(long long stride) { return (int)((4 * stride + kLeafBytes - 1) / kLeafBytes) + 1; }

int launch_hash_rows(const float* x, const PartEntry* table, uint32_t* leaves, unsigned char* out,
                     long long stride, int rows_per_part, int rows, cudaStream_t st)
{
    HashArgs a{x, table, leaves, out, stride, rows_per_part, rows, hash_max_leaves(stride)};
    const long long threads = (long long)rows * a.max_leaves;
    hash_leaves_kernel<<<(unsigned)((threads + 127) / 128), 128, 0, st>>>(a);
    hash_roots_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, st>>>(a);
    BTARD_CUDA_TRY(cudaGetLastError());
    count_launch(2);
    return BTARD_OK;
}

}  // namespace btard
