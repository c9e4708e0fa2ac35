// hash.cuh -- the bucket and sign hash functions of the Count Sketch (Algorithm 4 line 2), device side.
//
//   h_j(i) = ((a_j*i + b_j) mod p) mod c,   s_j(i) = 2*(((a'_j*i + b'_j) mod p) & 1) - 1,   p = 2^31-1.
//
// All arithmetic is integer and exact.  Three facts are used to keep it cheap:
//   * x mod p for x < 2^62 folds twice (2^31 = 1 mod p) and subtracts p at most once;
//   * consecutive coordinates differ by a_j before the reduction, so a thread that owns a run of
//     coordinates pays the 64-bit product once and one add + conditional subtract afterwards;
//   * "mod c" is a mask when c is a power of two, otherwise a multiply-high by a precomputed
//     reciprocal with one correction (exact for every y < 2^31, proven in make_bucketizer below).
#pragma once
#include <stdint.h>

namespace ssgd {

constexpr uint32_t P31 = 0x7FFFFFFFu;
constexpr int MAX_R = 15;

struct HashRow { uint32_t a, b, a2, b2; };
struct HashParams { HashRow row[MAX_R]; };  // 240 bytes, passed to kernels by value

struct Bucketizer {
    uint32_t c;      // number of columns
    uint32_t mask;   // c - 1 when c is a power of two
    uint32_t magic;  // floor(2^(31+L) / c), L = ceil(log2 c), when c is not a power of two
    uint32_t shift;  // L - 1
};

// Host: reciprocal for y mod c, y < 2^31, 1 <= c < 2^31.
// With 2^(L-1) < c < 2^L and m = floor(2^(31+L)/c) (2^31 <= m < 2^32):
//   y*m / 2^(31+L) = y/c - y*eps/2^(31+L) with 0 <= eps < 1 and y < 2^31, so the error is < 2^-L < 1
//   and q' = floor(y*m / 2^(31+L)) is floor(y/c) or one less; the remainder y - q'*c lies in [0, 2c).
inline Bucketizer make_bucketizer(uint64_t c) {
    Bucketizer bk{};
    bk.c = (uint32_t)c;
    if ((c & (c - 1)) == 0) { bk.mask = (uint32_t)(c - 1); return bk; }
    uint32_t L = 0;
    while ((1ull << L) < c) ++L;
    bk.magic = (uint32_t)((1ull << (31 + L)) / c);
    bk.shift = L - 1;
    return bk;
}

#ifdef __CUDACC__

// Programmatic dependent launch: every kernel of the step lets its successor's blocks become resident
// early (trigger) and waits for its predecessor to finish and flush before it touches global memory
// (wait).  Both are no-ops when the launch does not carry the attribute.  Every block must reach
// pdl_wait() before it exits, so that "kernel N finished" always implies "kernel N-1 finished".
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// x mod (2^31-1) for x < 2^62 + 2^31.
__device__ __forceinline__ uint32_t mod_p31(uint64_t x) {
    const uint32_t lo = (uint32_t)x & P31;
    const uint32_t hi = (uint32_t)(x >> 31);          // < 2^31 + 1
    const uint32_t s = lo + hi;                       // < 2^32
    uint32_t t = (s & P31) + (s >> 31);               // <= 2^31
    if (t >= P31) t -= P31;
    return t;
}

// (a*i + b) mod p
__device__ __forceinline__ uint32_t lin_hash(uint32_t a, uint32_t b, uint32_t i) {
    return mod_p31((uint64_t)a * (uint64_t)i + (uint64_t)b);
}

// ((a*i + b) mod p  +  a) mod p  =  (a*(i+1) + b) mod p
__device__ __forceinline__ uint32_t next_hash(uint32_t y, uint32_t a) {
    uint32_t t = y + a;                               // < 2p < 2^32
    if (t >= P31) t -= P31;
    return t;
}

template <bool POW2>
__device__ __forceinline__ uint32_t bucket_of(uint32_t y, const Bucketizer& bk) {
    if (POW2) return y & bk.mask;
    const uint32_t q = __umulhi(y, bk.magic) >> bk.shift;
    uint32_t rem = y - q * bk.c;
    if (rem >= bk.c) rem -= bk.c;
    return rem;
}

// Bucket and sign of NC consecutive coordinates i0 .. i0+NC-1 in row j.
// hb[e] = bucket | (sign bit << 31): bit 31 SET means s = -1 (low bit of the sign hash is 0).
template <bool POW2, int NC>
__device__ __forceinline__ void row_hashes(const HashRow& hr, const Bucketizer& bk, uint32_t i0,
                                           uint32_t (&hb)[NC]) {
    uint32_t y = lin_hash(hr.a, hr.b, i0);
    uint32_t z = lin_hash(hr.a2, hr.b2, i0);
#pragma unroll
    for (int e = 0; e < NC; ++e) {
        hb[e] = bucket_of<POW2>(y, bk) | ((~z & 1u) << 31);
        if (e + 1 < NC) { y = next_hash(y, hr.a); z = next_hash(z, hr.a2); }
    }
}

__device__ __forceinline__ float apply_sign(float x, uint32_t hb) {
    return __uint_as_float(__float_as_uint(x) ^ (hb & 0x80000000u));  // x * s_j(i), exact
}

#endif  // __CUDACC__
}  // namespace ssgd
