// rr_fill: buf[i] = low 32 bits of sm64(i).  The read path needs a region whose contents are a
// known function of the address so that checksums prove which lines were read (the paper's
// benchmark, Section 2.1, does not care about contents).  Write-bandwidth bound: each thread
// hashes four consecutive word indices and stores them as one 16-byte streaming store, a warp
// covering 512 contiguous bytes per store.
#include "rr_device.cuh"
#include "rr_internal.h"

namespace rr {

__global__ void __launch_bounds__(256) fill_kernel(uint4 *__restrict__ buf, uint64_t n_vec,
                                                   uint32_t *__restrict__ tail_dst,
                                                   uint64_t tail_first, uint32_t tail_words)
{
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n_vec; k += stride) {
        const uint64_t i = k << 2;
        uint4 w;
        w.x = (uint32_t)sm64(i);
        w.y = (uint32_t)sm64(i + 1);
        w.z = (uint32_t)sm64(i + 2);
        w.w = (uint32_t)sm64(i + 3);
        __stcs(buf + k, w);
    }
    if (blockIdx.x == 0 && threadIdx.x < tail_words)
        tail_dst[threadIdx.x] = (uint32_t)sm64(tail_first + threadIdx.x);
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
    const uint64_t n_vec = n_words >> 2;
    const uint32_t tail = (uint32_t)(n_words & 3u);
    uint64_t blocks = (n_vec + 255) / 256;
    const uint64_t cap = (uint64_t)f.nsm * 8;  // 2048 resident threads per SM
    if (blocks > cap) blocks = cap;
    if (blocks == 0) blocks = 1;
    rr::fill_kernel<<<(uint32_t)blocks, 256, 0, (cudaStream_t)stream>>>(
        (uint4 *)buf, n_vec, (uint32_t *)buf + (n_vec << 2), n_vec << 2, tail);
    RR_CUDA(cudaGetLastError());
    return RR_OK;
}
