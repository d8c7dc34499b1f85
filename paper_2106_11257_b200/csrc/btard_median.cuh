// Coordinate-wise median in registers: order-preserving integer keys and a comparator network.
#pragma once
#include <cstdint>

namespace btard {

// Batcher's odd-even merge sort as a comparator network on registers (N a power of two).  All
// indices are compile-time constants, so when only the middle outputs are used the compiler drops
// every comparator that does not feed them.
template <int N, typename T = int>
struct OddEvenNetwork {
    template <int LO, int CNT, int R>
    static __device__ __forceinline__ void merge(T (&k)[N])
    {
        constexpr int STEP = R * 2;
        if constexpr (STEP < CNT) {
            merge<LO, CNT, STEP>(k);
            merge<LO + R, CNT, STEP>(k);
#pragma unroll
            for (int i = LO + R; i + R < LO + CNT; i += STEP) {
                const T lo = min(k[i], k[i + R]), hi = max(k[i], k[i + R]);
                k[i] = lo;
                k[i + R] = hi;
            }
        } else {
            const T lo = min(k[LO], k[LO + R]), hi = max(k[LO], k[LO + R]);
            k[LO] = lo;
            k[LO + R] = hi;
        }
    }
    template <int LO, int CNT>
    static __device__ __forceinline__ void sort(T (&k)[N])
    {
        if constexpr (CNT > 1) {
            sort<LO, CNT / 2>(k);
            sort<LO + CNT / 2, CNT / 2>(k);
            merge<LO, CNT, 1>(k);
        }
    }
};

// Signed-integer image of a float whose integer order is the IEEE total order of the floats.
__device__ __forceinline__ int signed_key(float f)
{
    const int b = __float_as_int(f);
    return b ^ ((b >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float signed_key_value(int k)
{
    return __int_as_float(k ^ ((k >> 31) & 0x7fffffff));
}


// Median of the first n of N2 values held by one thread (n == N2 when EXACT: the two middle outputs are
// fixed registers and the network is pruned to them; otherwise the unused inputs hold the largest key and
// the middle is picked at run time).  Even n: the mean of the two middle values, formed in fp64.
template <int N2, bool EXACT>
__device__ __forceinline__ float median_of_keys(int (&key)[N2], int n)
{
    OddEvenNetwork<N2>::template sort<0, N2>(key);
    int ka = 0, kb = 0;
    if (EXACT) {
        ka = key[(N2 - 1) / 2];
        kb = key[N2 / 2];
    } else {
        const int ia = (n - 1) >> 1, ib = n >> 1;      // no dynamic register indexing
#pragma unroll
        for (int i = 0; i < N2; ++i) {
            if (i == ia) ka = key[i];
            if (i == ib) kb = key[i];
        }
    }
    return (float)(((double)signed_key_value(ka) + (double)signed_key_value(kb)) * 0.5);
}

// The same median on the values themselves, for columns without a NaN: among such values the order of
// the floats is the order of their keys (up to the sign of a zero, which no sum can see), so the key
// conversion of every input is saved.  Unused inputs (i >= n) must hold +infinity.
template <int N2, bool EXACT>
__device__ __forceinline__ float median_of_values(float (&x)[N2], int n)
{
    OddEvenNetwork<N2, float>::template sort<0, N2>(x);
    float a = 0.f, b = 0.f;
    if (EXACT) {
        a = x[(N2 - 1) / 2];
        b = x[N2 / 2];
    } else {
        const int ia = (n - 1) >> 1, ib = n >> 1;      // no dynamic register indexing
#pragma unroll
        for (int i = 0; i < N2; ++i) {
            if (i == ia) a = x[i];
            if (i == ib) b = x[i];
        }
    }
    return (float)(((double)a + (double)b) * 0.5);
}

}  // namespace btard
