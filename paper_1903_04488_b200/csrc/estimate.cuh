// estimate.cuh -- Algorithm 4 estimate(i): the median of the r signed buckets of a coordinate.
#pragma once
#include <stdint.h>

namespace ssgd {
#ifdef __CUDACC__

__device__ __forceinline__ float table_load(const float* p) { return __ldg(p); }

__device__ __forceinline__ void cswap(float& a, float& b) {
    const float lo = fminf(a, b), hi = fmaxf(a, b);
    a = lo; b = hi;
}

template <int R>
__device__ __forceinline__ float median_of(float (&a)[R]) {
    if constexpr (R == 1) {
        return a[0];
    } else if constexpr (R == 3) {
        return fmaxf(fminf(a[0], a[1]), fminf(fmaxf(a[0], a[1]), a[2]));
    } else if constexpr (R == 5) {
        // sort two pairs; the smaller of the two minima and the larger of the two maxima cannot be
        // the median; the median of the remaining three is the median of five
        cswap(a[0], a[1]); cswap(a[3], a[4]);
        const float lo = fmaxf(a[0], a[3]);   // larger of the pair minima
        const float hi = fminf(a[1], a[4]);   // smaller of the pair maxima
        return fmaxf(fminf(lo, hi), fminf(fmaxf(lo, hi), a[2]));
    } else {
        // general odd R: odd-even transposition sort in registers, then the middle element
#pragma unroll
        for (int round = 0; round < R; ++round)
#pragma unroll
            for (int p = round & 1; p + 1 < R; p += 2) cswap(a[p], a[p + 1]);
        return a[R / 2];
    }
}

#endif  // __CUDACC__
}  // namespace ssgd
