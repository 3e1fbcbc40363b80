// Device-side helpers of librr (sm_100a): the hash, the exact remainder by a window length,
// special registers, cache-bypassing vector loads.
#pragma once
#include <cstdint>

namespace rr {

constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;

// First output of a SplitMix64 generator whose state is x.
__host__ __device__ __forceinline__ uint64_t sm64(uint64_t x)
{
    uint64_t z = x + kGamma;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Exact r mod n for n < 2^32 with one high multiply: m = floor((2^64-1)/n) gives a quotient
// estimate that is the true quotient or one less, so one conditional subtraction finishes it.
struct Divisor {
    uint64_t m;
    uint32_t n;
};
__host__ __device__ __forceinline__ Divisor make_divisor(uint32_t n)
{
    Divisor d;
    d.n = n;
    d.m = 0xFFFFFFFFFFFFFFFFull / n;
    return d;
}
__device__ __forceinline__ uint32_t mod_exact(uint64_t r, const Divisor &d)
{
    uint64_t q = __umul64hi(r, d.m);
    uint64_t rem = r - q * d.n;
    if (rem >= d.n) rem -= d.n;
    return (uint32_t)rem;
}

__device__ __forceinline__ uint32_t smid()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t nsmid()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%nsmid;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint64_t globaltimer()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// One lane's share of a coalesced line: W consecutive 32-bit words through the read-only path,
// not allocated in L1.  Not volatile: the region is constant for the kernel's lifetime, so the
// compiler may hoist these above the arithmetic of earlier reads.
template <int W>
__device__ __forceinline__ void load_lane(const void *p, uint32_t (&d)[W]);

template <>
__device__ __forceinline__ void load_lane<1>(const void *p, uint32_t (&d)[1])
{
    asm("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(d[0]) : "l"(p));
}
template <>
__device__ __forceinline__ void load_lane<2>(const void *p, uint32_t (&d)[2])
{
    asm("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(d[0]), "=r"(d[1]) : "l"(p));
}
template <>
__device__ __forceinline__ void load_lane<4>(const void *p, uint32_t (&d)[4])
{
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "l"(p));
}

}  // namespace rr
