// Host-only parts of librr: status strings, device facts, the window policy and the reach rule.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <functional>
#include <mutex>
#include <utility>
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

__global__ void nsmid_kernel(uint32_t *out) { *out = nsmid(); }

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

extern "C" int32_t rr_device_info(rr_device_info_t *out, void *scratch_dev, void *stream_)
{
    if (!out) return RR_ERR_ARG;
    if (scratch_dev && (uintptr_t)scratch_dev % 16u) return RR_ERR_ALIGN;
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
    if (prop.major == 10 && scratch_dev) {  // the one-thread kernel exists for sm_100a only
        cudaStream_t stream = (cudaStream_t)stream_;
        uint32_t h = 0;
        rr::nsmid_kernel<<<1, 1, 0, stream>>>((uint32_t *)scratch_dev);
        RR_CUDA(cudaGetLastError());
        RR_CUDA(cudaMemcpyAsync(&h, scratch_dev, sizeof(h), cudaMemcpyDeviceToHost, stream));
        RR_CUDA(cudaStreamSynchronize(stream));
        out->nsm_reg = h;
    }
    return RR_OK;
}

extern "C" int32_t rr_make_windows(uint64_t region_bytes, uint32_t W, uint64_t window_bytes,
                                   uint32_t n_groups, uint32_t policy, uint64_t seed,
                                   rr_window_t *out, double *coverage)
{
    if (!(W == 1 || W == 2 || W == 4) || n_groups == 0 || n_groups > RR_MAX_GROUPS || policy > 2 ||
        !out)
        return RR_ERR_ARG;
    const uint64_t line = 128ull * W;
    const uint64_t L = region_bytes / line;
    if (L == 0 || L > 0xFFFFFFFFull) return RR_ERR_RANGE;
    const uint64_t S = std::min(std::max<uint64_t>(window_bytes / line, 1), L);
    if (policy == 2) {  // overlapping windows of S lines, first at 0, last ending at L
        uint64_t reached = 0, covered = 0;  // lines below `reached` have been accounted for
        for (uint32_t g = 0; g < n_groups; ++g) {
            const uint64_t base = n_groups > 1 ? (uint64_t)g * (L - S) / (n_groups - 1) : 0;
            out[g].base_line = (uint32_t)base;
            out[g].n_lines = (uint32_t)S;
            const uint64_t end = base + S;
            if (end > reached) {
                covered += end - std::max(base, reached);
                reached = end;
            }
        }
        if (coverage) *coverage = (double)covered / (double)L;
        return RR_OK;
    }
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

// ---- host-only policy rules that decide the plan a run uses ---------------------------------

extern "C" int32_t rr_reach_next(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                                 uint64_t step_bytes, uint64_t *next_size)
{
    if (!next_size || step_bytes == 0) return RR_ERR_ARG;
    double plateau = 0;
    uint64_t good = 0;
    const int32_t cliff = rr_reach(size_bytes, gbps, n_points, &plateau, &good);
    if (cliff < 0) return cliff;
    *next_size = 0;
    if (!cliff) return 0;
    const uint64_t *above = std::upper_bound(size_bytes, size_bytes + n_points, good);
    if (above == size_bytes + n_points) return 0;
    const uint64_t bad = *above;
    if (bad - good <= step_bytes) return 0;
    const uint64_t mid = ((good + bad) / 2) / step_bytes * step_bytes;
    if (mid <= good || mid >= bad) return 0;
    *next_size = mid;
    return 1;
}

extern "C" int32_t rr_sm_reach(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                               double keep, uint64_t *reach_bytes)
{
    if (!size_bytes || !gbps || !reach_bytes || n_points == 0 || !(keep > 0.0) || keep > 1.0)
        return RR_ERR_ARG;
    if (std::adjacent_find(size_bytes, size_bytes + n_points, std::greater_equal<uint64_t>()) !=
        size_bytes + n_points)
        return RR_ERR_ARG;
    double level = gbps[0];
    if (n_points >= 3) {
        double first[3] = {gbps[0], gbps[1], gbps[2]};
        std::sort(first, first + 3);
        level = first[1];
    }
    uint64_t reach = size_bytes[0];
    for (uint32_t k = 0; k < n_points && gbps[k] >= keep * level; ++k) reach = size_bytes[k];
    *reach_bytes = reach;
    return RR_OK;
}

extern "C" int32_t rr_owner_map(const uint16_t *group_of_sm, uint32_t nsm, uint16_t *owner_of_sm,
                                uint32_t *n_owners)
{
    if (!group_of_sm || !owner_of_sm || !n_owners || nsm == 0 || nsm > RR_MAX_SM) return RR_ERR_ARG;
    std::vector<uint32_t> order;
    for (uint32_t s = 0; s < nsm; ++s)
        if (group_of_sm[s] != RR_SM_INACTIVE) order.push_back(s);
    std::stable_sort(order.begin(), order.end(),
                     [&](uint32_t a, uint32_t b) { return group_of_sm[a] < group_of_sm[b]; });
    std::fill(owner_of_sm, owner_of_sm + nsm, (uint16_t)RR_SM_INACTIVE);
    for (size_t k = 0; k < order.size(); ++k) owner_of_sm[order[k]] = (uint16_t)k;
    *n_owners = (uint32_t)order.size();
    return RR_OK;
}

extern "C" int32_t rr_phase_window(uint64_t slice_bytes, uint64_t sm_reach_bytes, uint32_t max_parts,
                                   uint32_t *parts, uint64_t *sub_bytes)
{
    if (!parts || !sub_bytes || slice_bytes == 0 || sm_reach_bytes == 0 || max_parts == 0)
        return RR_ERR_ARG;
    typedef unsigned __int128 u128;
    uint32_t q = 1;
    for (; q < max_parts; q *= 2)
        if ((u128)slice_bytes * 4 <= (u128)sm_reach_bytes * q) break;  // slice/q <= reach/4
    *parts = q;
    *sub_bytes = slice_bytes / q + (slice_bytes % q ? 1 : 0);
    return RR_OK;
}

extern "C" int32_t rr_rebalance_weights(const uint32_t *work, const uint64_t *finish_ns,
                                        uint32_t n_groups, uint32_t scale, uint32_t *weight)
{
    if (!work || !finish_ns || !weight || n_groups == 0 || n_groups > RR_MAX_GROUPS || scale == 0)
        return RR_ERR_ARG;
    typedef unsigned __int128 u128;
    const u128 none = ~(u128)0;
    std::vector<u128> rate(n_groups, 0);
    u128 slowest = none;
    for (uint32_t g = 0; g < n_groups; ++g)
        if (finish_ns[g] && work[g]) {
            rate[g] = std::max<u128>(1, ((u128)work[g] << 48) / finish_ns[g]);
            slowest = std::min(slowest, rate[g]);
        }
    if (slowest == none) return RR_ERR_RANGE;  // nobody finished anything
    const u128 token = std::max<u128>(1, slowest >> 10);
    u128 total = 0;
    for (u128 &r : rate) {
        if (!r) r = token;
        total += r;
    }
    for (uint32_t g = 0; g < n_groups; ++g)
        weight[g] = (uint32_t)std::max<u128>(1, (rate[g] * scale + total / 2) / total);
    return RR_OK;
}

extern "C" int32_t rr_group_finish(const uint64_t *t_start, const uint64_t *t_end,
                                   const uint16_t *group_of_sm, uint32_t nsm, uint32_t n_groups,
                                   uint64_t *finish_ns, uint64_t *span_ns)
{
    if (!t_start || !t_end || !group_of_sm || !finish_ns || !span_ns || nsm == 0 ||
        nsm > RR_MAX_SM || n_groups == 0 || n_groups > RR_MAX_GROUPS)
        return RR_ERR_ARG;
    uint64_t begin = ~0ull, last = 0;
    for (uint32_t s = 0; s < nsm; ++s)
        if (t_end[s]) {
            begin = std::min(begin, t_start[s]);
            last = std::max(last, t_end[s]);
        }
    std::fill(finish_ns, finish_ns + n_groups, 0ull);
    *span_ns = last ? last - begin : 0;
    for (uint32_t s = 0; s < nsm; ++s) {
        const uint32_t g = group_of_sm[s];
        if (!t_end[s] || g == RR_SM_INACTIVE) continue;
        if (g >= n_groups) return RR_ERR_MAP;
        finish_ns[g] = std::max<uint64_t>(finish_ns[g], t_end[s] > begin ? t_end[s] - begin : 1);
    }
    return RR_OK;
}

extern "C" int32_t rr_finish_spread_ppm(const uint64_t *finish_ns, uint32_t n_groups, uint32_t *ppm)
{
    if (!finish_ns || !ppm || n_groups == 0) return RR_ERR_ARG;
    uint64_t lo = ~0ull, hi = 0;
    for (uint32_t g = 0; g < n_groups; ++g)
        if (finish_ns[g]) {
            lo = std::min(lo, finish_ns[g]);
            hi = std::max(hi, finish_ns[g]);
        }
    *ppm = hi ? (uint32_t)(((unsigned __int128)(hi - lo) * 1000000u) / hi) : 0u;
    return RR_OK;
}

extern "C" int32_t rr_window_cover(const rr_window_t *windows, uint32_t n_groups, uint64_t n_lines,
                                   uint64_t *covered, uint32_t *depth_min, uint32_t *depth_max)
{
    if (!windows || !covered || !depth_min || !depth_max || n_groups == 0 ||
        n_groups > RR_MAX_GROUPS)
        return RR_ERR_ARG;
    // sweep line over (position, +1 / -1) events
    std::vector<std::pair<uint64_t, int>> ev;
    for (uint32_t g = 0; g < n_groups; ++g) {
        const uint64_t lo = windows[g].base_line, hi = lo + windows[g].n_lines;
        if (hi == lo || hi > n_lines) return RR_ERR_RANGE;
        ev.emplace_back(lo, +1);
        ev.emplace_back(hi, -1);
    }
    std::sort(ev.begin(), ev.end());
    uint64_t cov = 0, at = 0;
    int depth = 0;
    uint32_t dmin = ~0u, dmax = 0;
    for (size_t k = 0; k < ev.size();) {
        const uint64_t pos = ev[k].first;
        if (depth > 0 && pos > at) {
            cov += pos - at;
            dmin = std::min(dmin, (uint32_t)depth);
            dmax = std::max(dmax, (uint32_t)depth);
        }
        for (; k < ev.size() && ev[k].first == pos; ++k) depth += ev[k].second;
        at = pos;
    }
    *covered = cov;
    *depth_min = dmin == ~0u ? 0 : dmin;
    *depth_max = dmax;
    return RR_OK;
}
