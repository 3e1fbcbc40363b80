// Host-side internals of librr: scratch layout, CUDA error capture, launch geometry.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "rr.h"

namespace rr {

// ---- device scratch layout (rr_scratch_bytes) -------------------------------------------
constexpr uint32_t kMaxBlocksPerSm = 2;
constexpr uint32_t kMaxRecords = RR_MAX_SM * kMaxBlocksPerSm;

struct BlockRecord {      // one per block that did work
    uint32_t smid;
    uint32_t slot;        // 0-based claim order on that SM (PER_SM) / blockIdx (LOGICAL)
    uint64_t t_start;     // %globaltimer, ns
    uint64_t t_end;
};

struct ProbeRecord {      // one per probe launch
    uint64_t t_start[2];
    uint64_t t_end[2];
    uint32_t claim[2];
    uint32_t ready;       // chosen SMs that have arrived at the common start
    uint32_t gave_up;     // chosen SMs that stopped waiting for the other one
    uint32_t done_warps[2];            // warps of each SM that have finished their fixed share
    unsigned long long extra_lines[2]; // lines each SM read beyond its share, waiting for the other
    uint32_t sink;        // never read: keeps the extra loads observable
    uint32_t pad;
};
static_assert(sizeof(ProbeRecord) % 16 == 0, "records are packed in an array");

struct ScratchHeader {
    uint32_t status;
    uint32_t violations;
    uint32_t blocks_run;
    uint32_t pad;
    uint32_t claim[RR_MAX_SM];
    BlockRecord rec[kMaxRecords];
    ProbeRecord probe;
    unsigned long long pool_next[RR_MAX_GROUPS];  // POOLED: next work item of each group
};

// Bytes after the header used by rr_cluster (see rr_cluster.cu).
size_t cluster_scratch_bytes(uint32_t n);

// ---- error capture -------------------------------------------------------------------------
void set_cuda_error(cudaError_t e, const char *what);
#define RR_CUDA(call)                                   \
    do {                                                \
        cudaError_t e__ = (call);                       \
        if (e__ != cudaSuccess) {                       \
            ::rr::set_cuda_error(e__, #call);           \
            return RR_ERR_CUDA;                         \
        }                                               \
    } while (0)

// ---- device facts cached per device ---------------------------------------------------------
struct DeviceFacts {
    int device;
    int nsm;
    int cc_major, cc_minor;
    int smem_per_sm;
    int smem_per_block_optin;
};
int32_t device_facts(DeviceFacts *out);
uint64_t device_fact_queries();  // how often the runtime was really asked

}  // namespace rr
