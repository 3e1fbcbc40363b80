// rr_cluster: SM x SM pair-throughput matrix -> SM resource groups (paper Section 2.2, Fig. 3:
// the matrix is "rearranged" until groups show as diagonal blocks; here that is average-linkage
// agglomeration with a largest-gap cut).  One block of 1024 threads; everything that decides an
// integer is exact integer arithmetic, and every floating-point step is a single correctly
// rounded IEEE double operation (explicit _rn intrinsics, so nothing is contracted into an FMA).
#include <cmath>
#include <cstring>

#include "rr_internal.h"

namespace rr {

constexpr int kClusterThreads = 1024;

struct ClusterOut {
    uint32_t n_groups;
    uint32_t best_k;
    double confidence;
    double gap;
};

// Work arrays behind the scratch header, all sized for n SMs.
struct ClusterLayout {
    size_t off_T, off_keys, off_q, off_sum, off_h, off_group, off_out, total;
    uint32_t n, pairs, pow2;
    __host__ __device__ explicit ClusterLayout(uint32_t n_) : n(n_)
    {
        pairs = n * (n - 1) / 2;
        pow2 = 1;
        while (pow2 < pairs) pow2 <<= 1;
        size_t o = 0;
        auto take = [&](size_t bytes) {
            size_t at = o;
            o += (bytes + 15) & ~(size_t)15;
            return at;
        };
        off_T = take(sizeof(float) * n * n);
        off_keys = take(sizeof(uint64_t) * pow2);
        off_q = take(sizeof(uint32_t) * n * n);
        off_sum = take(sizeof(uint64_t) * n * n);
        off_h = take(sizeof(double) * n);
        off_group = take(sizeof(int32_t) * n);
        off_out = take(sizeof(ClusterOut));
        total = o;
    }
};

size_t cluster_scratch_bytes(uint32_t n) { return ClusterLayout(n).total; }

// In-place ascending bitonic sort of P (a power of two) 64-bit keys by one block.
__device__ void block_sort(uint64_t *keys, uint32_t P)
{
    for (uint32_t k = 2; k <= P; k <<= 1)
        for (uint32_t j = k >> 1; j > 0; j >>= 1) {
            for (uint32_t i = threadIdx.x; i < P; i += blockDim.x) {
                const uint32_t partner = i ^ j;
                if (partner > i) {
                    const uint64_t a = keys[i], b = keys[partner];
                    const bool ascending = (i & k) == 0;
                    if ((a > b) == ascending) {
                        keys[i] = b;
                        keys[partner] = a;
                    }
                }
            }
            __syncthreads();
        }
}

struct Candidate {
    uint64_t s;   // sum of q over the member pairs of clusters a and b
    uint32_t p;   // number of member pairs, size[a]*size[b]; 0 = no candidate
    uint32_t a, b;
};

// mean(x) < mean(y) by cross-multiplication; ties go to the lexicographically smaller (a,b).
__device__ __forceinline__ bool better(const Candidate &x, const Candidate &y)
{
    if (x.p == 0) return false;
    if (y.p == 0) return true;
    const uint64_t l = x.s * y.p, r = y.s * x.p;
    if (l != r) return l < r;
    return x.a < y.a || (x.a == y.a && x.b < y.b);
}

__device__ __forceinline__ Candidate shfl_down(const Candidate &c, int o)
{
    Candidate r;
    r.s = __shfl_down_sync(0xFFFFFFFFu, c.s, o);
    r.p = __shfl_down_sync(0xFFFFFFFFu, c.p, o);
    r.a = __shfl_down_sync(0xFFFFFFFFu, c.a, o);
    r.b = __shfl_down_sync(0xFFFFFFFFu, c.b, o);
    return r;
}

__global__ void __launch_bounds__(kClusterThreads, 1) cluster_kernel(uint8_t *work, uint32_t n, uint32_t flags)
{
    const ClusterLayout lay(n);
    const float *T = (const float *)(work + lay.off_T);
    uint64_t *keys = (uint64_t *)(work + lay.off_keys);
    uint32_t *q = (uint32_t *)(work + lay.off_q);
    uint64_t *sum = (uint64_t *)(work + lay.off_sum);
    double *h = (double *)(work + lay.off_h);
    int32_t *group = (int32_t *)(work + lay.off_group);
    ClusterOut *out = (ClusterOut *)(work + lay.off_out);

    __shared__ uint32_t size[RR_MAX_SM], alive[RR_MAX_SM], rep[RR_MAX_SM];
    __shared__ uint32_t merge_a[RR_MAX_SM], merge_b[RR_MAX_SM], merge_pairs[RR_MAX_SM];
    __shared__ Candidate warp_best[kClusterThreads / 32];
    __shared__ Candidate best;
    __shared__ uint32_t sh_count, sh_best_k, sh_pow2;
    __shared__ uint64_t sh_median;
    const uint32_t tid = threadIdx.x, nn = n * n;

    // 1. symmetrised off-diagonal entries, as sortable keys (positive doubles order like integers)
    auto sym = [&](uint32_t i, uint32_t j) {
        double s = __dmul_rn(__dadd_rn((double)T[i * n + j], (double)T[j * n + i]), 0.5);
        if (flags & RR_CLUSTER_SOLO_NORMALISE)  // pair rate relative to the two solo rates
            s = __ddiv_rn(s, __dadd_rn((double)T[i * n + i], (double)T[j * n + j]));
        return s;
    };
    for (uint32_t k = tid; k < lay.pow2; k += blockDim.x) keys[k] = ~0ull;
    __syncthreads();
    for (uint32_t idx = tid; idx < nn; idx += blockDim.x) {
        const uint32_t i = idx / n, j = idx % n;
        if (i < j) keys[i * n - i * (i + 1) / 2 + (j - i - 1)] = (uint64_t)__double_as_longlong(sym(i, j));
    }
    __syncthreads();
    block_sort(keys, lay.pow2);
    // 2. quantise against the lower median
    const double med = __longlong_as_double((long long)keys[(lay.pairs - 1) / 2]);
    for (uint32_t idx = tid; idx < nn; idx += blockDim.x) {
        const uint32_t i = idx / n, j = idx % n;
        uint32_t v = 0;
        if (i != j) {
            const double r = rint(__ddiv_rn(__dmul_rn(sym(i, j), 1048576.0), med));
            v = (r >= 4294967295.0) ? 0xFFFFFFFFu : (uint32_t)r;
        }
        q[idx] = v;
        sum[idx] = v;
    }
    for (uint32_t i = tid; i < n; i += blockDim.x) {
        size[i] = 1;
        alive[i] = 1;
    }
    __syncthreads();

    // 3. average linkage: n-1 merges
    for (uint32_t step = 0; step + 1 < n; ++step) {
        Candidate c;
        c.s = 0;
        c.p = 0;
        c.a = c.b = 0;
        for (uint32_t idx = tid; idx < nn; idx += blockDim.x) {
            const uint32_t a = idx / n, b = idx % n;
            if (a < b && alive[a] && alive[b]) {
                Candidate x;
                x.s = sum[idx];
                x.p = size[a] * size[b];
                x.a = a;
                x.b = b;
                if (better(x, c)) c = x;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const Candidate y = shfl_down(c, o);
            if (better(y, c)) c = y;
        }
        if ((tid & 31u) == 0) warp_best[tid >> 5] = c;
        __syncthreads();
        if (tid < 32) {
            c = warp_best[tid];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const Candidate y = shfl_down(c, o);
                if (better(y, c)) c = y;
            }
            if (tid == 0) {
                best = c;
                merge_a[step] = c.a;
                merge_b[step] = c.b;
                merge_pairs[step] = c.p;
                h[step] = __ddiv_rn((double)c.s, (double)c.p);
            }
        }
        __syncthreads();
        const uint32_t ba = best.a, bb = best.b;
        for (uint32_t k = tid; k < n; k += blockDim.x)
            if (alive[k] && k != ba && k != bb) {
                const uint64_t s = sum[ba * n + k] + sum[bb * n + k];
                sum[ba * n + k] = s;
                sum[k * n + ba] = s;
            }
        __syncthreads();
        if (tid == 0) {
            size[ba] += size[bb];
            alive[bb] = 0;
        }
        __syncthreads();
    }

    // 4. cut at the largest gap among cuts leaving 2 .. n/3 clusters (first maximum wins)
    if (tid == 0) {
        out->n_groups = 1;
        out->confidence = 0.0;
        out->gap = 0.0;
        out->best_k = 0;
        uint32_t best_k = 0;
        const uint32_t max_clusters = n / 3;
        if (max_clusters >= 2) {
            double best_gap = -1.0;
            for (uint32_t k = n - max_clusters; k <= n - 2; ++k) {
                const double gap = __dsub_rn(h[k], h[k - 1]);
                if (gap > best_gap) {
                    best_gap = gap;
                    best_k = k;
                }
            }
            out->gap = best_gap;
            out->best_k = best_k;
        }
        sh_best_k = best_k;
        sh_count = 0;
    }
    for (uint32_t i = tid; i < n; i += blockDim.x) group[i] = 0;
    __syncthreads();
    const uint32_t best_k = sh_best_k;
    if (best_k == 0) return;  // fewer than 6 SMs: no group level

    for (uint32_t i = tid; i < n; i += blockDim.x) {
        uint32_t r = i;
        for (uint32_t k = 0; k < best_k; ++k)
            if (r == merge_b[k]) r = merge_a[k];
        rep[i] = r;
    }
    __syncthreads();

    // 5. null rule: robust sigma of the q of pairs lying in different clusters
    for (uint32_t idx = tid; idx < nn; idx += blockDim.x) {
        const uint32_t i = idx / n, j = idx % n;
        if (i < j && rep[i] != rep[j]) keys[atomicAdd(&sh_count, 1u)] = q[idx];
    }
    __syncthreads();
    const uint32_t nb = sh_count;
    if (tid == 0) {
        uint32_t P = 1;
        while (P < nb) P <<= 1;
        sh_pow2 = P;
    }
    __syncthreads();
    const uint32_t P = sh_pow2;
    for (uint32_t k = nb + tid; k < P; k += blockDim.x) keys[k] = ~0ull;
    __syncthreads();
    block_sort(keys, P);
    if (tid == 0) sh_median = keys[(nb - 1) / 2];
    __syncthreads();
    const uint64_t bmed = sh_median;
    for (uint32_t k = tid; k < nb; k += blockDim.x) {
        const uint64_t x = keys[k];
        keys[k] = x > bmed ? x - bmed : bmed - x;
    }
    __syncthreads();
    block_sort(keys, P);
    if (tid == 0) {
        const double mad = (double)keys[(nb - 1) / 2];
        const double sigma = __ddiv_rn(__dmul_rn(1.4826, mad), __dsqrt_rn((double)merge_pairs[best_k]));
        const double gap = out->gap;
        const double conf = sigma > 0.0 ? __ddiv_rn(gap, sigma) : (gap > 0.0 ? INFINITY : 0.0);
        out->confidence = conf;
        // a gap below 1 % of the median pair rate (2^20 in these units) is background, not a group
        if (gap >= __dmul_rn(4.0, sigma) && gap >= 10485.76) {
            // 6. groups numbered by their smallest SM id (a cluster is named by its smallest member)
            uint32_t G = 0;
            for (uint32_t i = 0; i < n; ++i)
                if (rep[i] == i) merge_a[i] = G++;  // reuse: label of representative i
            for (uint32_t i = 0; i < n; ++i) group[i] = (int32_t)merge_a[rep[i]];
            out->n_groups = G;
        }
    }
}

}  // namespace rr

using namespace rr;

extern "C" int32_t rr_cluster(const float *T_host, uint32_t n, uint32_t flags, void *scratch_dev,
                              int32_t *group_of_sm_host, uint32_t *n_groups, double *confidence,
                              double *heights_host, void *stream_)
{
    if (!T_host || !scratch_dev || !group_of_sm_host || !n_groups || n < 2 || n > RR_MAX_SM ||
        flags > RR_CLUSTER_SOLO_NORMALISE)
        return RR_ERR_ARG;
    if ((uintptr_t)scratch_dev % 16u) return RR_ERR_ALIGN;
    for (uint32_t i = 0; i < n; ++i)
        for (uint32_t j = 0; j < n; ++j) {
            const float x = T_host[(size_t)i * n + j];
            if ((i != j || flags) && !(x > 0.0f && std::isfinite(x))) return RR_ERR_ARG;
        }
    DeviceFacts f;
    int32_t rc = device_facts(&f);
    if (rc != RR_OK) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    const ClusterLayout lay(n);
    uint8_t *work = (uint8_t *)scratch_dev + sizeof(ScratchHeader);
    RR_CUDA(cudaMemcpyAsync(work + lay.off_T, T_host, sizeof(float) * n * n, cudaMemcpyHostToDevice,
                            stream));
    cluster_kernel<<<1, kClusterThreads, 0, stream>>>(work, n, flags);
    RR_CUDA(cudaGetLastError());
    ClusterOut out;
    RR_CUDA(cudaMemcpyAsync(&out, work + lay.off_out, sizeof(out), cudaMemcpyDeviceToHost, stream));
    RR_CUDA(cudaMemcpyAsync(group_of_sm_host, work + lay.off_group, sizeof(int32_t) * n,
                            cudaMemcpyDeviceToHost, stream));
    if (heights_host)
        RR_CUDA(cudaMemcpyAsync(heights_host, work + lay.off_h, sizeof(double) * (n - 1),
                                cudaMemcpyDeviceToHost, stream));
    RR_CUDA(cudaStreamSynchronize(stream));
    *n_groups = out.n_groups;
    if (confidence) *confidence = out.confidence;
    return RR_OK;
}
