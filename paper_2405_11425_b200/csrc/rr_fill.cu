// rr_fill: buf[i] = low 32 bits of sm64(i).  The read path needs a region whose contents are a
// known function of the address so that checksums prove which lines were read (the paper's
// benchmark, Section 2.1, does not care about contents).
//
// The hash costs ~18 integer instructions per word, two thirds of them on the shift/logic pipe,
// which would hold the kernel at 0.69 of the write bandwidth.  Two things bring it to the store
// rate:
//  * Eight consecutive word indices per thread share most of the first hash step.  With
//    z = i + gamma, the words 8k .. 8k+7 are t + 0 .. t + 7 for t = 8k + gamma, and the low three
//    bits of t are those of gamma (101b): t + 0, 1, 2 change only the low three bits, t + 3 carries
//    once, and t + 3 .. t + 7 again differ only in the low three bits.  Inside such a run the
//    term z >> 30 and the high half of z ^ (z >> 30) are common, and the low half differs by a
//    constant XOR.  So step one costs four instructions per run plus one per word instead of six
//    per word.
//  * One 32-byte store per thread (st.global.cs.v8.b32), so that a warp writes 1 KiB of
//    consecutive bytes per store instruction.
#include "rr_device.cuh"
#include "rr_internal.h"

namespace rr {

constexpr uint64_t kMul1 = 0xBF58476D1CE4E5B9ull, kMul2 = 0x94D049BB133111EBull;

// The hash from the point where y = z ^ (z >> 30) is known.
__device__ __forceinline__ uint32_t hash_tail(uint64_t y)
{
    y *= kMul1;
    y ^= y >> 27;
    y *= kMul2;
    return (uint32_t)(y ^ (y >> 31));
}

// Words u + 0 .. u + count-1 where adding stays inside the low three bits of u (= n0).
template <int FIRST, int COUNT>
__device__ __forceinline__ void hash_run(uint64_t u, uint32_t n0, uint32_t (&out)[8])
{
    const uint64_t s = u >> 30;
    const uint32_t y_hi = (uint32_t)(u >> 32) ^ (uint32_t)(s >> 32);
    const uint32_t y_lo = (uint32_t)u ^ (uint32_t)s;
#pragma unroll
    for (int j = 0; j < COUNT; ++j) {
        const uint32_t flip = n0 ^ (n0 + (uint32_t)j);  // turns the low bits n0 into n0 + j
        out[FIRST + j] = hash_tail(((uint64_t)y_hi << 32) | (uint64_t)(y_lo ^ flip));
    }
}

__device__ __forceinline__ void store_256(uint32_t *dst, const uint32_t (&w)[8])
{
    asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst),
                 "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]),
                 "r"(w[7])
                 : "memory");
}

__global__ void __launch_bounds__(256) fill_kernel(uint32_t *__restrict__ buf, uint64_t n_chunks,
                                                   uint32_t tail_words)
{
    constexpr uint32_t n0 = (uint32_t)(kGamma & 7u);  // low three bits of every t below
    constexpr int kRunA = 8 - (int)n0;                // words before the carry
    static_assert(n0 != 0 && kRunA >= 1 && kRunA <= 7, "two runs per chunk");
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n_chunks; k += stride) {
        const uint64_t t = (k << 3) + kGamma;
        uint32_t w[8];
        hash_run<0, kRunA>(t, n0, w);
        hash_run<kRunA, 8 - kRunA>(t + kRunA, 0u, w);
        store_256(buf + (k << 3), w);
    }
    if (blockIdx.x == 0 && threadIdx.x < tail_words)  // fewer than eight words left over
        buf[(n_chunks << 3) + threadIdx.x] = (uint32_t)sm64((n_chunks << 3) + threadIdx.x);
}

}  // namespace rr

extern "C" int32_t rr_fill(void *buf, uint64_t n_words, void *stream)
{
    if (n_words == 0) return RR_OK;
    if (!buf) return RR_ERR_ARG;
    if ((uintptr_t)buf % 512u) return RR_ERR_ALIGN;
    if (n_words > (1ull << 40)) return RR_ERR_RANGE;
    rr::DeviceFacts f;
    int32_t rc = rr::device_facts(&f);
    if (rc != RR_OK) return rc;
    const uint64_t n_chunks = n_words >> 3;
    const uint32_t tail = (uint32_t)(n_words & 7u);
    uint64_t blocks = (n_chunks + 255) / 256;
    const uint64_t cap = (uint64_t)f.nsm * 8;  // 2048 resident threads per SM
    if (blocks > cap) blocks = cap;
    if (blocks == 0) blocks = 1;
    rr::fill_kernel<<<(uint32_t)blocks, 256, 0, (cudaStream_t)stream>>>((uint32_t *)buf, n_chunks,
                                                                         tail);
    RR_CUDA(cudaGetLastError());
    return RR_OK;
}
