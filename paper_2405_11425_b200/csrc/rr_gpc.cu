// rr_gpc_map: an independent look at the SM layout through thread-block-cluster placement.
// The paper (Section 1.1) notes that a program cannot ask which GPC an SM is on, and finds its
// groups by timing alone (Section 2.2).  Blocks of one cluster are always co-scheduled on one GPC,
// so launching clusters and recording %smid per block yields "same GPC" facts with no timing
// noise: SMs that ever appear in one cluster are merged (union-find on the host).  Every
// contention group found by the probe should nest inside one of these GPCs.
#include <numeric>
#include <vector>

#include "rr_device.cuh"
#include "rr_internal.h"

namespace rr {

__global__ void gpc_map_kernel(uint32_t *smid_of_block, uint32_t spin_ns)
{
    if (threadIdx.x == 0) {
        smid_of_block[blockIdx.x] = smid();
        // stay resident for a moment so that later clusters land on other SMs (bounded wait)
        const uint64_t t0 = globaltimer();
        for (int it = 0; it < 4096 && globaltimer() - t0 < spin_ns; ++it) __nanosleep(64);
    }
}

constexpr uint32_t kGpcMaxBlocks = 4096;

}  // namespace rr

using namespace rr;

extern "C" int32_t rr_gpc_map(void *scratch_dev, int32_t *gpc_of_sm_host, uint32_t *n_gpcs,
                              uint32_t nsm, void *stream_)
{
    if (!scratch_dev || !gpc_of_sm_host || !n_gpcs || nsm == 0 || nsm > RR_MAX_SM)
        return RR_ERR_ARG;
    if ((uintptr_t)scratch_dev % 16u) return RR_ERR_ALIGN;
    DeviceFacts f;
    int32_t rc = device_facts(&f);
    if (rc != RR_OK) return rc;
    if (nsm != (uint32_t)f.nsm) return RR_ERR_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    uint32_t *dev = (uint32_t *)((char *)scratch_dev + sizeof(ScratchHeader));
    std::vector<uint32_t> parent(nsm);
    std::iota(parent.begin(), parent.end(), 0u);
    auto find = [&](uint32_t x) {
        while (parent[x] != x) x = parent[x] = parent[parent[x]];
        return x;
    };
    std::vector<uint32_t> host(kGpcMaxBlocks);
    // cluster sizes 2..8 (portable), with a big and a small shared-memory footprint so that the
    // scheduler packs clusters differently; a few rounds each
    for (uint32_t csize = 2; csize <= 8; ++csize) {
        for (int heavy = 0; heavy < 2; ++heavy) {
            const size_t smem = heavy ? 100 * 1024 : 0;
            if (heavy)
                RR_CUDA(cudaFuncSetAttribute(gpc_map_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem));
            uint32_t blocks = ((heavy ? 2u : 8u) * nsm / csize) * csize;
            if (blocks > kGpcMaxBlocks) blocks = (kGpcMaxBlocks / csize) * csize;
            RR_CUDA(cudaMemsetAsync(dev, 0xFF, sizeof(uint32_t) * blocks, stream));
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(blocks);
            cfg.blockDim = dim3(32);
            cfg.dynamicSmemBytes = smem;
            cfg.stream = stream;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = csize;
            attr.val.clusterDim.y = 1;
            attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            RR_CUDA(cudaLaunchKernelEx(&cfg, gpc_map_kernel, dev, 20000u));
            RR_CUDA(cudaMemcpyAsync(host.data(), dev, sizeof(uint32_t) * blocks,
                                    cudaMemcpyDeviceToHost, stream));
            RR_CUDA(cudaStreamSynchronize(stream));
            for (uint32_t c = 0; c < blocks / csize; ++c) {
                const uint32_t first = host[c * csize];
                if (first >= nsm) continue;
                for (uint32_t k = 1; k < csize; ++k) {
                    const uint32_t s = host[c * csize + k];
                    if (s >= nsm) continue;
                    const uint32_t a = find(first), b = find(s);
                    if (a != b) parent[std::max(a, b)] = std::min(a, b);
                }
            }
        }
    }
    // an SM that never hosted a block of any cluster simply stays a component of its own
    // canonical labels: GPCs numbered by their smallest SM id
    std::vector<int32_t> label(nsm, -1);
    uint32_t G = 0;
    for (uint32_t s = 0; s < nsm; ++s) {
        const uint32_t r = find(s);
        if (label[r] < 0) label[r] = (int32_t)G++;
        gpc_of_sm_host[s] = label[r];
    }
    *n_gpcs = G;
    return RR_OK;
}
