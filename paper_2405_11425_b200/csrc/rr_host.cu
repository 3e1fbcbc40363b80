// Host-only parts of librr: status strings, device facts, the window policy and the reach rule.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "rr_device.cuh"
#include "rr_internal.h"

namespace rr {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e, const char *what)
{
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", what, cudaGetErrorString(e),
                  cudaGetErrorName(e));
    cudaGetLastError();  // clear the sticky-less error state
}

// Facts of each device are asked of the runtime once and kept: they cannot change while the
// process lives, and six attribute queries per launch are visible next to a 2 ms kernel.
static std::mutex g_facts_mutex;
static DeviceFacts g_facts[64];
static bool g_facts_known[64];
static std::atomic<uint64_t> g_n_fact_queries{0};

uint64_t device_fact_queries() { return g_n_fact_queries.load(); }

int32_t device_facts(DeviceFacts *out)
{
    int dev = 0;
    RR_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return RR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_facts_mutex);
    if (!g_facts_known[dev]) {
        DeviceFacts f;
        f.device = dev;
        g_n_fact_queries.fetch_add(1);
        RR_CUDA(cudaDeviceGetAttribute(&f.nsm, cudaDevAttrMultiProcessorCount, dev));
        RR_CUDA(cudaDeviceGetAttribute(&f.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
        RR_CUDA(cudaDeviceGetAttribute(&f.cc_minor, cudaDevAttrComputeCapabilityMinor, dev));
        RR_CUDA(cudaDeviceGetAttribute(&f.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor,
                                       dev));
        RR_CUDA(cudaDeviceGetAttribute(&f.smem_per_block_optin,
                                       cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        g_facts[dev] = f;
        g_facts_known[dev] = true;
    }
    *out = g_facts[dev];
    if (out->cc_major != 10) {
        std::snprintf(g_cuda_error, sizeof(g_cuda_error),
                      "device has compute capability %d.%d; this library holds sm_100a code only",
                      out->cc_major, out->cc_minor);
        return RR_ERR_UNSUPPORTED;
    }
    if (out->nsm > (int)RR_MAX_SM) return RR_ERR_UNSUPPORTED;
    return RR_OK;
}

__device__ uint32_t g_nsmid;
__global__ void nsmid_kernel() { g_nsmid = nsmid(); }

}  // namespace rr

extern "C" const char *rr_strerror(int32_t code)
{
    switch (code) {
        case RR_OK: return "ok";
        case RR_ERR_ARG: return "invalid argument";
        case RR_ERR_ALIGN: return "pointer not aligned (buffer 512 B, output 8 B, scratch 16 B)";
        case RR_ERR_RANGE: return "size out of range (region, line count or window)";
        case RR_ERR_MAP: return "SM-to-group map is inconsistent";
        case RR_ERR_CUDA: return "CUDA call failed (see rr_last_cuda_error)";
        case RR_ERR_SM_UNCOVERED: return "an active SM never received a block";
        case RR_ERR_TIMEOUT: return "device-side wait ran out";
        case RR_ERR_CHECK: return "checked variant rejected an address";
        case RR_ERR_UNSUPPORTED: return "unsupported device";
        case RR_ERR_STATIC_LIMIT:
            return "request exceeds the built-in scratch of rr_random_read_static "
                   "(at most 192 SMs)";
        default: return "unknown status";
    }
}

extern "C" const char *rr_last_cuda_error(void) { return rr::g_cuda_error; }

extern "C" size_t rr_scratch_bytes(void)
{
    return sizeof(rr::ScratchHeader) + rr::cluster_scratch_bytes(RR_MAX_SM);
}

extern "C" int32_t rr_device_info(rr_device_info_t *out)
{
    if (!out) return RR_ERR_ARG;
    std::memset(out, 0, sizeof(*out));
    int dev = 0;
    RR_CUDA(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    RR_CUDA(cudaGetDeviceProperties(&prop, dev));
    out->nsm_prop = (uint32_t)prop.multiProcessorCount;
    out->cc_major = (uint32_t)prop.major;
    out->cc_minor = (uint32_t)prop.minor;
    size_t fr = 0, tot = 0;
    RR_CUDA(cudaMemGetInfo(&fr, &tot));
    out->free_bytes = fr;
    out->total_bytes = tot;
    int clk = 0, bus = 0;
    RR_CUDA(cudaDeviceGetAttribute(&clk, cudaDevAttrMemoryClockRate, dev));
    RR_CUDA(cudaDeviceGetAttribute(&bus, cudaDevAttrGlobalMemoryBusWidth, dev));
    out->mem_clock_khz = (uint32_t)clk;
    out->bus_width_bits = (uint32_t)bus;
    out->l2_bytes = (uint64_t)prop.l2CacheSize;
    out->smem_per_sm = (uint32_t)prop.sharedMemPerMultiprocessor;
    out->smem_per_block_optin = (uint32_t)prop.sharedMemPerBlockOptin;
    out->theoretical_gbps = 2.0 * (double)clk * 1e3 * (double)bus / 8.0 * 1e-9;
    std::snprintf(out->name, sizeof(out->name), "%s", prop.name);
    for (int i = 0; i < 16; ++i)
        std::snprintf(out->uuid + 2 * i, 3, "%02x", (unsigned)(unsigned char)prop.uuid.bytes[i]);
    if (prop.major == 10) {  // the one-thread kernel exists for sm_100a only
        uint32_t h = 0;
        rr::nsmid_kernel<<<1, 1>>>();
        RR_CUDA(cudaMemcpyFromSymbol(&h, rr::g_nsmid, sizeof(h)));
        out->nsm_reg = h;
    }
    return RR_OK;
}

extern "C" int32_t rr_make_windows(uint64_t region_bytes, uint32_t W, uint64_t window_bytes,
                                   uint32_t n_groups, uint32_t policy, uint64_t seed,
                                   rr_window_t *out, double *coverage)
{
    if (!(W == 1 || W == 2 || W == 4) || n_groups == 0 || n_groups > RR_MAX_GROUPS || policy > 1 ||
        !out)
        return RR_ERR_ARG;
    const uint64_t line = 128ull * W;
    const uint64_t L = region_bytes / line;
    if (L == 0 || L > 0xFFFFFFFFull) return RR_ERR_RANGE;
    const uint64_t S = std::min(std::max<uint64_t>(window_bytes / line, 1), L);
    const uint64_t K = (L + S - 1) / S;
    const uint64_t chunk = L / K;
    std::vector<bool> used(K, false);
    for (uint32_t g = 0; g < n_groups; ++g) {
        const uint64_t c = policy ? rr::sm64(seed ^ (uint64_t)g) % K : g % K;
        out[g].base_line = (uint32_t)(c * chunk);
        out[g].n_lines = (uint32_t)((c + 1 == K ? L : (c + 1) * chunk) - c * chunk);
        used[c] = true;
    }
    if (coverage) *coverage = (double)std::count(used.begin(), used.end(), true) / (double)K;
    return RR_OK;
}

extern "C" int32_t rr_make_weighted_windows(uint64_t region_bytes, uint32_t W, uint32_t n_groups,
                                            const uint32_t *weight, uint32_t n_warps,
                                            uint64_t max_window_bytes, rr_window_t *out,
                                            uint32_t *warp_start)
{
    if (!(W == 1 || W == 2 || W == 4) || n_groups == 0 || n_groups > RR_MAX_GROUPS || !weight ||
        !out || !warp_start || n_warps == 0)
        return RR_ERR_ARG;
    const uint64_t line = 128ull * W;
    const uint64_t L = region_bytes / line;
    if (L == 0 || L > 0xFFFFFFFFull) return RR_ERR_RANGE;
    uint64_t total = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        if (weight[g] == 0) return RR_ERR_ARG;
        total += weight[g];
    }
    if (total > 0xFFFFFFFFull) return RR_ERR_RANGE;  // L * prefix and V * prefix stay in 64 bits
    uint64_t prefix = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        const uint64_t next = prefix + weight[g];
        const uint64_t lo = L * prefix / total, hi = L * next / total;
        const uint64_t vlo = (uint64_t)n_warps * prefix / total, vhi = (uint64_t)n_warps * next / total;
        if (hi == lo || vhi == vlo) return RR_ERR_RANGE;
        if (max_window_bytes && (hi - lo) * line > max_window_bytes) return RR_ERR_RANGE;
        out[g].base_line = (uint32_t)lo;
        out[g].n_lines = (uint32_t)(hi - lo);
        warp_start[g] = (uint32_t)vlo;
        prefix = next;
    }
    warp_start[n_groups] = n_warps;
    return RR_OK;
}

extern "C" int32_t rr_reach(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                            double *plateau, uint64_t *reach_bytes)
{
    if (!size_bytes || !gbps || !plateau || !reach_bytes || n_points == 0) return RR_ERR_ARG;
    const uint64_t lo = 4ull << 30, hi = 32ull << 30;
    std::vector<double> mid;
    for (uint32_t k = 0; k < n_points; ++k) {
        if (k && size_bytes[k] <= size_bytes[k - 1]) return RR_ERR_ARG;
        if (size_bytes[k] >= lo && size_bytes[k] <= hi) mid.push_back(gbps[k]);
    }
    if (mid.empty()) return RR_ERR_RANGE;
    std::sort(mid.begin(), mid.end());
    const double P = mid[(mid.size() - 1) / 2];
    *plateau = P;
    uint32_t first_bad = n_points;
    for (uint32_t k = 0; k < n_points && first_bad == n_points; ++k)
        if (size_bytes[k] > hi && gbps[k] < 0.8 * P) first_bad = k;
    *reach_bytes = 0;
    for (uint32_t k = 0; k < first_bad; ++k)
        if (gbps[k] >= 0.9 * P) *reach_bytes = size_bytes[k];
    return first_bad != n_points ? 1 : 0;
}
