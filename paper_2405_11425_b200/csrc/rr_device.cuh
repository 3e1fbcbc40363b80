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
// HINT = 0: no L2 prefetch qualifier; 128 / 256: ld ... .L2::128B / .L2::256B, which ask L2 to
// bring in the aligned 128- / 256-byte block around the address.
#define RR_LD_LANE(HINT_, QUAL_)                                                                  \
    template <>                                                                                   \
    __device__ __forceinline__ void load_lane<1, HINT_>(const void *p, uint32_t (&d)[1])          \
    {                                                                                             \
        asm("ld.global.nc.L1::no_allocate" QUAL_ ".u32 %0, [%1];" : "=r"(d[0]) : "l"(p));         \
    }                                                                                             \
    template <>                                                                                   \
    __device__ __forceinline__ void load_lane<2, HINT_>(const void *p, uint32_t (&d)[2])          \
    {                                                                                             \
        asm("ld.global.nc.L1::no_allocate" QUAL_ ".v2.u32 {%0, %1}, [%2];"                        \
            : "=r"(d[0]), "=r"(d[1])                                                              \
            : "l"(p));                                                                            \
    }                                                                                             \
    template <>                                                                                   \
    __device__ __forceinline__ void load_lane<4, HINT_>(const void *p, uint32_t (&d)[4])          \
    {                                                                                             \
        asm("ld.global.nc.L1::no_allocate" QUAL_ ".v4.u32 {%0, %1, %2, %3}, [%4];"                \
            : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])                                      \
            : "l"(p));                                                                            \
    }

template <int W, int HINT = 0>
__device__ __forceinline__ void load_lane(const void *p, uint32_t (&d)[W]);
RR_LD_LANE(0, "")
RR_LD_LANE(128, ".L2::128B")
RR_LD_LANE(256, ".L2::256B")
#undef RR_LD_LANE

// ---- bulk-copy staging: one thread asks the copy engine for a whole line ------------------------
// cp.async.bulk global -> this block's shared memory, completion counted in bytes on an mbarrier.
// Source and destination 16-byte aligned, size a multiple of 16.  Never multicast, never a peer's
// memory: the source is the caller's region on this GPU.
__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes,
                                          uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            dst_smem),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
// One poll of the barrier's phase; true once the phase with this parity has completed.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void lds_lane(uint32_t addr, uint32_t (&d)[1])
{
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(d[0]) : "r"(addr));
}
__device__ __forceinline__ void lds_lane(uint32_t addr, uint32_t (&d)[2])
{
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(d[0]), "=r"(d[1]) : "r"(addr));
}
__device__ __forceinline__ void lds_lane(uint32_t addr, uint32_t (&d)[4])
{
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(addr));
}

}  // namespace rr
