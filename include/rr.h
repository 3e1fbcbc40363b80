/*
 * rr.h -- C ABI of librr: warp-coalesced random cache-line reads over the whole HBM with
 * SM resource groups held to address windows (arXiv 2405.11425, written for B200 / sm_100a).
 *
 * Conventions that hold for every entry point
 *   - extern "C"; plain pointers and sizes.  Each pointer is marked DEVICE or HOST below.
 *   - Every function returns an int32_t status: RR_OK (0) or a negative RR_ERR_* code.  Nothing
 *     throws, aborts or exits.  rr_strerror() names a code; rr_last_cuda_error() gives the text
 *     of the last CUDA failure seen by the calling thread (for RR_ERR_CUDA).
 *   - The caller owns all device memory (region buffer, outputs, scratch).  Unless an entry
 *     point says otherwise the library allocates nothing on the device and keeps no state
 *     between calls.  Host arrays are borrowed for the duration of the call only.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Arguments are validated on the host before any CUDA call: a call that returns RR_ERR_ARG,
 *     RR_ERR_ALIGN, RR_ERR_RANGE or RR_ERR_MAP has launched nothing.
 *   - Units: a "word" is 32 bits; a "line" is 128*W bytes (W = words per lane = 1, 2 or 4),
 *     aligned to its own size, counted from the start of the buffer; GB/s = 1e9 bytes/s.
 *
 * Definitions shared by several entry points (the paper gives prose only; these are the
 * readings this library implements)
 *   sm64(x)      = first output of a SplitMix64 generator whose state is x (add
 *                  0x9E3779B97F4A7C15, then the 30/27/31 xor-shift-multiply finaliser)
 *   word(i)      = low 32 bits of sm64(i)                  -- contents of buffer word i
 *   k_v          = sm64(sm64(seed) ^ v)                    -- key of logical warp v
 *   r(seed,v,i)  = sm64(k_v + i * 0x9E3779B97F4A7C15)      -- i-th draw of warp v
 *   line(v,i)    = base + (r mod n)   for a window of n lines starting at line `base`
 *                  (RR_INDEX_STRIDE: base + ((i * V + v) mod n), V = warps in the call)
 *                  (RR_INDEX_MIXED, period k: read i with i mod k == 0 is read i/k of the warp's
 *                  sequential walk, base + (((i/k) * V + v) mod n); other reads are random)
 *                  (RR_INDEX_PHASED: the window is cut into Q = ceil(n / sub) sub-windows
 *                  [floor(n q / Q), floor(n (q+1) / Q)), sub = phase_window_bytes / (128 W);
 *                  read i belongs to phase p = floor(i / phase_reads) and draws
 *                  base + lo_q + (r mod (hi_q - lo_q)) with q = (p + stagger) mod Q, where
 *                  stagger = floor(smid * Q / nsm) in RR_MODE_PER_SM and 0 otherwise)
 *   checksum     = {X, S}: X = xor, S = sum mod 2^32 of every 32-bit word the warp read
 */
#ifndef RR_H_
#define RR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ---- */
#define RR_OK 0
#define RR_ERR_ARG (-1)          /* NULL / out-of-domain argument                               */
#define RR_ERR_ALIGN (-2)        /* buffer not 512-byte aligned, output not 8-byte aligned      */
#define RR_ERR_RANGE (-3)        /* region shorter than a line, >= 2^32 lines, window past end  */
#define RR_ERR_MAP (-4)          /* SM->group map names a group >= n_groups, or no SM is active */
#define RR_ERR_CUDA (-5)         /* a CUDA call failed; see rr_last_cuda_error()                */
#define RR_ERR_SM_UNCOVERED (-6) /* an active SM never received a block                         */
#define RR_ERR_TIMEOUT (-7)      /* reserved: a bounded device-side wait ran out                */
#define RR_ERR_CHECK (-8)        /* checked variant saw an address outside its window; the      */
                                 /* offending loads were skipped                                */
#define RR_ERR_UNSUPPORTED (-9)  /* device is not the one this library was built for            */
#define RR_ERR_STATIC_LIMIT (-10) /* rr_random_read_static: request exceeds its built-in scratch */

/* ---- limits ---- */
#define RR_MAX_SM 256u      /* SM ids the tables can hold (B200 has 148)                       */
#define RR_MAX_GROUPS 256u  /* one window per group; the naive control uses one group per SM   */
#define RR_MAX_WARPS_PER_SM 32u /* one 1024-thread block per SM                                 */
#define RR_SM_INACTIVE 0xFFFFu

/* ---- enums (plain integers in the structs) ---- */
#define RR_MODE_LOGICAL 0u /* v = global warp index 0..n_warps-1, window = whole region        */
#define RR_MODE_PER_SM 1u  /* v = smid * warps_per_sm + warp, window by SM group               */
#define RR_MODE_POOLED 2u  /* logical warps owned by SM groups; the group's SMs share the work  */
#define RR_INDEX_RANDOM 0u
#define RR_INDEX_STRIDE 1u
#define RR_INDEX_PHASED 2u /* random inside a sub-window that moves with the read counter         */
#define RR_INDEX_MIXED 3u  /* every mix_period-th read sequential, the others random              */
#define RR_VARIANT_LDG 0u         /* ld.global.nc.L1::no_allocate vector loads                  */
#define RR_VARIANT_LDG_CHECKED 1u /* same, every address bounds-checked before the load         */
#define RR_VARIANT_PACKED 2u      /* every lane loads 16 bytes: one warp load covers 4/W lines  */
                                  /* (same lines and words; fewer instructions per line)        */
#define RR_VARIANT_SORTED 3u      /* RR_VARIANT_PACKED with each warp's reads taken in an order */
                                  /* that keeps the SM inside one part of its window at a time  */

const char *rr_strerror(int32_t code);
const char *rr_last_cuda_error(void);

/* ---- host-side bookkeeping the library keeps ----------------------------------------------
 * Three small caches live in the library for the life of the process, none of them on the
 * device: the attributes of each device (asked once), the launch configuration of each
 * (device, kernel, block size, blocks per SM) -- the dynamic shared-memory request that keeps one
 * block per SM, found by an occupancy search -- and two timing events per host thread and
 * device.  A repeated call therefore makes no attribute, occupancy or event-creation call.
 * rr_host_counters reports how often each of those runtime calls was really made (HOST struct);
 * it exists so that a test can see the caches work.                                            */
typedef struct {
    uint64_t occupancy_queries;   /* cudaOccupancyMaxActiveBlocksPerMultiprocessor calls         */
    uint64_t attribute_sets;      /* cudaFuncSetAttribute calls                                  */
    uint64_t event_creates;       /* cudaEventCreate calls                                       */
    uint64_t device_fact_queries; /* rounds of cudaDeviceGetAttribute queries                    */
} rr_host_counters_t;
int32_t rr_host_counters(rr_host_counters_t *out /*HOST*/);

/* ---- device facts ------------------------------------------------------------------------
 * Paper, Section 1.1: the %smid / %nsmid registers are the only layout facts a program gets.
 * Fills *out (HOST) for the current device.  nsm_reg is %nsmid, read by a one-thread kernel that
 * runs on `stream` and writes its answer into the first word of scratch_dev (DEVICE, 16-byte
 * aligned, at least 4 bytes; rr_scratch_bytes() will do); with scratch_dev == NULL nothing is
 * launched and nsm_reg stays 0.  Synchronises `stream` when it launches.
 * theoretical_gbps = 2 * memory clock * bus width / 8.                                        */
typedef struct {
    uint32_t nsm_prop;       /* cudaDeviceProp::multiProcessorCount                            */
    uint32_t nsm_reg;        /* %nsmid                                                         */
    uint32_t cc_major, cc_minor;
    uint64_t free_bytes, total_bytes;
    uint32_t mem_clock_khz, bus_width_bits;
    uint64_t l2_bytes;
    uint32_t smem_per_sm, smem_per_block_optin;
    double theoretical_gbps;
    char name[64];
    char uuid[40];           /* 32 hex digits, NUL-terminated                                  */
} rr_device_info_t;
int32_t rr_device_info(rr_device_info_t *out /*HOST*/, void *scratch_dev /*DEVICE or NULL*/,
                       void *stream);

/* ---- scratch ------------------------------------------------------------------------------
 * Bytes of DEVICE scratch rr_random_read / rr_probe_pair / rr_cluster need (claim table,
 * status words, per-block timing records, clustering work arrays).  16-byte aligned.  The
 * library clears what must start at zero; the contents after a call are what
 * rr_read_report() decodes.  One scratch buffer must not be shared by calls that overlap.    */
size_t rr_scratch_bytes(void);

/* ---- fill ---------------------------------------------------------------------------------
 * buf[i] = word(i) for i in [0, n_words).  buf: DEVICE, 512-byte aligned, n_words*4 bytes.
 * Asynchronous on `stream`.  n_words = 0 is a no-op.                                          */
int32_t rr_fill(void *buf /*DEVICE*/, uint64_t n_words, void *stream);

/* ---- random line reads -------------------------------------------------------------------
 * Paper, Section 2.1, Fig. 1 (the basic benchmark: each warp fetches whole lines of 32 words at
 * random positions of a region whose size is varied; 32-, 64- and 128-bit words), Section 2.1
 * second experiment and Section 2.4, Fig. 6 (all warps of an SM / of an SM group read inside
 * one chunk).
 *
 * The region is the prefix [0, region_bytes) of buf; L = floor(region_bytes / (128*W)) lines.
 * RR_MODE_LOGICAL: n_warps logical warps, each reading the whole region; any block may run
 *   any warp; out has n_warps entries.  With windows[n_groups] (HOST) and no group_of_sm, warp v
 *   reads inside windows[v mod n_groups] instead: a window chosen per warp with no regard for SMs
 *   -- the naive control of Section 2.1 one level finer than per SM (use rr_make_windows
 *   policy 1 for the windows).
 * RR_MODE_PER_SM: a persistent grid, warps_per_sm warps on every SM; a block reads %smid,
 *   claims the SM, looks its group and window up in a table in shared memory; warp
 *   v = smid*warps_per_sm + w.  group_of_sm == NULL: every SM active, window = whole region.
 *   Otherwise group_of_sm[nsm] (HOST) gives each SM's group or RR_SM_INACTIVE, and
 *   windows[n_groups] (HOST) the window of each group.  out has nsm*warps_per_sm entries;
 *   inactive SMs' entries are {0,0}.  nsm must equal the device's SM count (0 = take it).
 * RR_MODE_POOLED (Section 2.3 shows that a group's throughput belongs to the group, not to its
 *   SMs): n_warps logical warps; group g owns warps warp_start[g] .. warp_start[g+1]-1 (HOST
 *   array of n_groups+1 entries, warp_start[0] = 0, warp_start[n_groups] = n_warps) and they
 *   read inside windows[g].  The group's work is the line of its warps' reads; the persistent
 *   blocks of the group's SMs (warps_per_sm physical warps each) grab runs of that line from a
 *   per-group counter -- long runs at first, never shorter than pool_block_reads at the end --
 *   until it is used up (a group of one SM is simply split into equal shares, one per warp).  A group with more SMs then does not do more work than its shared
 *   translation path can carry, and no group becomes the straggler when warp_start follows the
 *   groups' capacities (rr_make_weighted_windows).  out has n_warps entries, accumulated with
 *   atomics (the call clears it first); the checksums do not depend on which SM did what.
 *   Every group that owns warps needs at least one active SM, else RR_ERR_MAP.
 * RR_INDEX_PHASED (LOGICAL and PER_SM modes; first_read must be a multiple of 32): Section 1.3
 *   wants each warp held to a smaller region; here that region also moves, so that an SM whose
 *   own translation cache is smaller than its share of memory works through its window one
 *   sub-window at a time while a whole cycle of phases still covers the window uniformly.
 *   SMs that share a window (the whole region when group_of_sm is NULL) start their cycles at
 *   staggered sub-windows, so the region can also be read from every SM with no partition.
 * RR_INDEX_MIXED (LOGICAL and PER_SM modes; Section 2.1 closes on sequential access being the
 *   faster kind): a blend of the two, one read in mix_period sequential, to place a workload
 *   between the random rate and the sequential ceiling.  mix_period = 1 is RR_INDEX_STRIDE.
 * RR_VARIANT_SORTED (W = 1, 2; RR_INDEX_RANDOM): the checksums do not depend on the order of a
 *   warp's reads, so the kernel is free to choose one.  This variant cuts the stream into epochs
 *   of sort_parts * sort_reads reads and performs the reads of an epoch part by part of the
 *   warp's window (sort_parts equal parts): at any moment an SM then works inside 1/sort_parts of
 *   its window, which its own translation cache can hold, although the window -- the set of lines
 *   the warp may read, Section 1.3 -- is unchanged and static.  Results are those of
 *   RR_VARIANT_PACKED bit for bit; the price is a second hash per read (one pass classifies the
 *   epoch's reads by part, then each part's reads are hashed again as full vectors) and
 *   5.25 KB of shared memory per warp.
 * Reads i in [first_read, first_read + reads_per_warp) of each warp's stream are performed
 * (reads_per_warp = 0 is valid: all checksums {0,0}).
 * unroll: independent loads kept in flight per warp: 0 (= default 8) or 2, 4, 8, 16, lowered
 *   so that unroll * W <= 32 (the ring lives in registers).  RR_VARIANT_PACKED counts warp
 *   loads of 4/W lines each (1, 2, 4 or 8; default 4), RR_VARIANT_SORTED likewise (1, 2 or 4;
 *   default 1, which measured fastest: the order already shortens the latency to be covered).
 *
 * out_dev (DEVICE, 8-byte aligned): pairs {X, S} of uint32.  scratch_dev: rr_scratch_bytes().
 * res == NULL: asynchronous on `stream`, no timing; decode the scratch later with
 *   rr_read_report().  res != NULL: the call records events around the launch, synchronises
 *   the stream, checks SM coverage and the status word, and fills *res (HOST).               */
typedef struct {
    uint32_t base_line, n_lines;
} rr_window_t;

typedef struct {
    const void *buf;            /* DEVICE, 512-byte aligned                                    */
    uint64_t region_bytes;
    uint32_t words_per_lane;    /* W: 1, 2, 4                                                  */
    uint32_t mode;              /* RR_MODE_*                                                   */
    uint32_t index_mode;        /* RR_INDEX_*                                                  */
    uint32_t n_warps;           /* LOGICAL, POOLED: number of logical warps                    */
    uint32_t warps_per_sm;      /* PER_SM, POOLED: 1..RR_MAX_WARPS_PER_SM (one block per SM)   */
    uint32_t nsm;               /* PER_SM, POOLED: SM count of the device, 0 = query           */
    uint64_t reads_per_warp;
    uint64_t first_read;
    uint64_t seed;
    const uint16_t *group_of_sm; /* HOST [nsm] or NULL                                         */
    const rr_window_t *windows;  /* HOST [n_groups] or NULL                                    */
    uint32_t n_groups;
    uint32_t variant;           /* RR_VARIANT_*                                                */
    uint32_t unroll;
    uint32_t pool_block_reads;  /* POOLED: smallest grab in reads, 0 = 64; else must be 0      */
    const uint32_t *warp_start; /* POOLED: HOST [n_groups+1]; else NULL                        */
    uint32_t phase_reads;       /* RR_INDEX_PHASED: reads per phase, a power of two >= 32      */
    uint32_t mix_period;        /* RR_INDEX_MIXED: a power of two in [1, 2^20]; else must be 0  */
    uint64_t phase_window_bytes; /* RR_INDEX_PHASED: largest sub-window                        */
    uint32_t sort_parts;        /* RR_VARIANT_SORTED: parts of the window: 2, 4, 8 or 16         */
    uint32_t sort_reads;        /* RR_VARIANT_SORTED: reads per part and epoch, a multiple of  */
                                /* 32 with sort_parts * sort_reads <= 4096 (16 x 256 is a good */
                                /* value); both 0 for every other variant                      */
} rr_read_params_t;

typedef struct {
    double seconds_event;   /* CUDA events around the launch (0 when not timed)                */
    double seconds_device;  /* max block end - min block start, %globaltimer                   */
    uint64_t bytes;         /* (active or logical) warps * reads_per_warp * 128 * W            */
    double gbps;            /* bytes / seconds_event / 1e9 (seconds_device when not timed)     */
    uint32_t status;        /* device status word: 0 = clean                                   */
    uint32_t violations;    /* checked variant: addresses rejected                             */
    uint32_t sms_covered;   /* PER_SM: active SMs that ran their warps                         */
    uint32_t blocks_run;    /* blocks that did work                                            */
} rr_result_t;

int32_t rr_random_read(const rr_read_params_t *params /*HOST*/, void *out_dev /*DEVICE*/,
                       void *scratch_dev /*DEVICE*/, rr_result_t *res /*HOST or NULL*/,
                       void *stream);

/* Decodes the scratch of the last rr_random_read that used it (call after the stream has
 * been synchronised; this function synchronises `stream` itself first).  Returns
 * RR_ERR_SM_UNCOVERED / RR_ERR_CHECK like the timed form of rr_random_read.                   */
int32_t rr_read_report(const rr_read_params_t *params /*HOST*/, const void *scratch_dev,
                       rr_result_t *res /*HOST*/, void *stream);

/* Start and end of every SM's block in the last rr_random_read that used this scratch
 * (%globaltimer, ns; both 0 for an SM that ran no block).  RR_MODE_PER_SM / RR_MODE_POOLED only.
 * t_start_host, t_end_host: HOST [nsm].  Synchronises `stream` first.  With these a caller can
 * see which SM group finished last and shift work between groups (Section 2.3).               */
int32_t rr_read_block_times(const void *scratch_dev /*DEVICE*/, uint32_t nsm,
                            uint64_t *t_start_host, uint64_t *t_end_host, void *stream);

/* ---- random line reads for callers that cannot allocate device memory ----------------------
 * (The paper has no counterpart: this is a packaging variant of rr_random_read.)
 *
 * Some callers have no way to hand the library a scratch buffer: code running inside another
 * framework's memory pool that may not call cudaMalloc, a plugin loaded after the host
 * application has claimed all device memory, or a hook that runs where allocation is forbidden.
 * For them this entry point performs exactly the read rr_random_read performs, but keeps the
 * claim table, status words and per-block timing records in a fixed array that is part of the
 * library image (RR_STATIC_SCRATCH_BYTES bytes, resident on every GPU that loads the library,
 * until the process exits).  It allocates no device memory -- no cudaMalloc, cudaFree or other
 * allocating CUDA or library routine is called (the launch-configuration cache above lives in
 * host memory) -- and creates no events:
 * res->seconds_event is 0 and res->gbps is computed from the device-side timers.
 *
 * Limit: at most RR_STATIC_MAX_SM SMs (the device's count, or the nsm passed in), and no
 * RR_MODE_POOLED (its work counters do not fit); both return RR_ERR_STATIC_LIMIT before
 * launching.  All other arguments, outputs and
 * status codes are those of rr_random_read (the caller still passes buf and out_dev).
 *
 * The first call on each device looks up the device address of the built-in array (the device
 * must be current); make that first call outside any stream capture.  Every call on a device
 * shares the one array, which still holds the previous call's contents, and clears it before
 * launching; two calls that overlap on the GPU (for instance on different streams) therefore
 * race on it: keep calls on one device in stream order.  res == NULL queues the work and
 * returns without waiting.                                                                    */
#define RR_STATIC_MAX_SM 192u
#define RR_STATIC_SCRATCH_BYTES 5888u
int32_t rr_random_read_static(const rr_read_params_t *params /*HOST*/, void *out_dev /*DEVICE*/,
                              rr_result_t *res /*HOST or NULL*/, void *stream);

/* ---- two-SM contention probe ---------------------------------------------------------------
 * Paper, Section 2.2, Fig. 2: the read kernel is run on two SMs only; a pair that shares a
 * translation resource is expected to lose throughput.  A full grid is launched; blocks exit
 * unless they are the first block on sm_a or sm_b.  Each surviving SM performs total_reads/2
 * random 128-byte line reads (W = 1) over the whole region with warps_per_sm warps (1..32;
 * total_reads must be a multiple of 2*warps_per_sm), warp ids and streams as in RR_MODE_PER_SM.
 * sm_a == sm_b: a solo run (total_reads/2 reads on that one SM).
 * The two blocks of a pair start together (the first waits at most 0.2 ms for the other), and a
 * warp that has finished its share keeps reading its stream, 32 reads at a time, until every
 * warp of the other SM has finished too (at most as many reads again): SMs differ in speed, and
 * a tail in which one runs alone would dilute the contention being measured.
 * out_dev: 2*warps_per_sm pairs {X,S} over the fixed share only: sm_a's warps, then sm_b's (zeros
 * for a solo run).
 * Synchronous.  res->bytes counts every line read (share and extra); res->gbps = those bytes /
 * (latest end - earliest start, %globaltimer);
 * res->seconds_event is the event time of the launch.  RR_ERR_SM_UNCOVERED if, after three
 * launches with growing grids, one of the SMs never received a block.                        */
int32_t rr_probe_pair(const void *buf /*DEVICE*/, uint64_t region_bytes, uint32_t sm_a,
                      uint32_t sm_b, uint64_t total_reads, uint32_t warps_per_sm, uint64_t seed,
                      void *out_dev /*DEVICE*/, void *scratch_dev /*DEVICE*/,
                      rr_result_t *res /*HOST*/, void *stream);

/* Bytes of DEVICE scratch rr_probe_matrix needs for nsm SMs (one timing record per pair).    */
size_t rr_probe_matrix_scratch_bytes(uint32_t nsm);

/* All unordered pairs and all solos: T_host[a*nsm+b] = T_host[b*nsm+a] = pair GB/s (median of
 * `repeats` sweeps, repeats >= 1), T_host[a*nsm+a] = solo GB/s.  Launches are queued back to
 * back per sweep and read back once.  out_dev as in rr_probe_pair (overwritten by every pair).
 *
 * The two SMs of a pair must read side by side for the figure to mean contention, so (i) they
 * start together and read until both are done (see rr_probe_pair), and
 * (ii) a pair whose overlap fraction
 *   (earliest end - latest start) / (latest end - earliest start)
 * is below 0.98 is measured again on its own with twice the reads, up to three doublings and
 * only while a doubling still raises the overlap by 0.01 (two SMs of different speed never
 * reach 0.98 however long they run); the sample with the best overlap is kept.
 * stats (HOST, may be NULL): the smallest kept overlap, how many pairs stayed below 0.98 in
 * some sweep, how many extra launches the rule cost.  overlap_host (HOST nsm*nsm float, may be
 * NULL): per pair, the smallest kept overlap over the sweeps (diagonal 1).                    */
typedef struct {
    double overlap_min;        /* smallest kept overlap over all pairs and sweeps              */
    uint32_t pairs_below_goal; /* pairs whose kept overlap stayed below 0.98 in some sweep     */
    uint32_t reruns;           /* extra launches with more reads                               */
    uint32_t relaunched;       /* pairs redone because an SM got no block in the queued launch */
} rr_probe_stats_t;
int32_t rr_probe_matrix(const void *buf /*DEVICE*/, uint64_t region_bytes, uint64_t total_reads,
                        uint32_t warps_per_sm, uint64_t seed, uint32_t repeats,
                        float *T_host /*HOST nsm*nsm*/, uint32_t nsm, void *out_dev /*DEVICE*/,
                        void *scratch_dev /*DEVICE*/, rr_probe_stats_t *stats /*HOST*/,
                        float *overlap_host /*HOST*/, void *stream);

/* The same for rows [row_begin, row_end) of the matrix only: pairs (a, b) with a in the range and
 * b >= a; the entries (a, b), (b, a) and (a, a) of T_host (and overlap_host) are written, the rest
 * left alone; stats cover these rows.  A caller can so probe a card in blocks of rows and keep
 * what is done (the full sweep takes ~10^4 launches).  rr_probe_matrix is rows [0, nsm).       */
int32_t rr_probe_rows(const void *buf /*DEVICE*/, uint64_t region_bytes, uint64_t total_reads,
                      uint32_t warps_per_sm, uint64_t seed, uint32_t repeats, uint32_t row_begin,
                      uint32_t row_end, float *T_host /*HOST nsm*nsm*/, uint32_t nsm,
                      void *out_dev /*DEVICE*/, void *scratch_dev /*DEVICE*/,
                      rr_probe_stats_t *stats /*HOST*/, float *overlap_host /*HOST*/, void *stream);

/* The rule that turns one probe's timers into a rate (host only).  t_start, t_end (ns), claim and
 * extra_lines hold one entry per SM (two for a pair, the first only when solo = 1); an SM with
 * claim 0 or no end time never ran: RR_ERR_SM_UNCOVERED.  gbps = bytes of the SMs that ran
 * (total_reads/2 + extra_lines[i] lines of 128 bytes each) / (latest end - earliest start);
 * overlap as defined above (1 for a solo run).                                                */
int32_t rr_probe_rate(const uint64_t *t_start, const uint64_t *t_end, const uint32_t *claim,
                      const uint64_t *extra_lines, uint32_t solo, uint64_t total_reads,
                      double *gbps, double *seconds, double *overlap);

/* ---- contention matrix -> SM groups --------------------------------------------------------
 * Paper, Section 2.2 and Figure 3 (the SM indices are reordered until the groups show up as
 * blocks of the matrix).  Here:
 * symmetrise, quantise against the median, average-linkage agglomeration with exact integer
 * sums, cut at the largest height gap among cuts leaving 2..n/3 clusters, null rule (gap below
 * 4 robust standard deviations of the height, or below 1 % of the median pair rate -- the paper
 * sets the faint background pattern aside -- gives one group), groups numbered by their smallest
 * SM id.  Runs as one block on the device.
 * T_host: HOST n*n float32 row-major; off-diagonal entries must be finite and > 0, else
 * RR_ERR_ARG; 2 <= n <= RR_MAX_SM.  flags = 0: the diagonal is ignored.
 * flags = RR_CLUSTER_SOLO_NORMALISE: every pair entry is first divided by the sum of the two
 * SMs' solo rates on the diagonal (which must then be finite and > 0), so an SM that is slow
 * on its own does not look contended.  group_of_sm_host: HOST int32[n].
 * heights_host: HOST double[n-1] or NULL (merge heights).  Synchronous.                      */
#define RR_CLUSTER_SOLO_NORMALISE 1u
int32_t rr_cluster(const float *T_host, uint32_t n, uint32_t flags, void *scratch_dev /*DEVICE*/,
                   int32_t *group_of_sm_host, uint32_t *n_groups, double *confidence,
                   double *heights_host, void *stream);

/* ---- cross-check of the layout by cluster placement -----------------------------------------
 * Paper, Section 1.1: a program is not told which GPC an SM belongs to.  Blocks of
 * one thread-block cluster always run on one GPC, so this call launches clusters of 2..8 small
 * blocks, records %smid per block and merges SMs that shared a cluster: gpc_of_sm_host[nsm]
 * (HOST) receives a GPC label per SM (numbered by smallest SM id), *n_gpcs their count.  No
 * timing is involved; every contention group found by rr_cluster on a probe matrix should lie
 * inside one of these GPCs (Section 2.2 found groups finer than GPCs).  nsm = the device's SM
 * count.  Synchronous; uses rr_scratch_bytes() of scratch.  An SM that never hosted a block of
 * any cluster stays a component of its own (it carries no placement information).             */
int32_t rr_gpc_map(void *scratch_dev /*DEVICE*/, int32_t *gpc_of_sm_host /*HOST*/,
                   uint32_t *n_gpcs, uint32_t nsm, void *stream);

/* ---- windows per group (host only) -------------------------------------------------------
 * Paper, Section 1.3 (each group confined to a window below the reach; half of memory as the
 * simple case) and Section 2.4.  The L lines of the region are cut into K = ceil(L /
 * floor(window_bytes / (128*W))) chunks of floor(L/K) lines, the last running to L.
 * policy 0: group g takes chunk g mod K.  policy 1 (the paper's naive per-SM control; pass one
 * group per SM): chunk sm64(seed ^ g) mod K.  *coverage (may be NULL) = distinct chunks used / K.
 * policy 2 (Section 1.3 does not ask for disjoint windows): n_groups windows of exactly
 * S = floor(window_bytes / (128*W)) lines (clipped to [1, L]), evenly spaced and overlapping:
 * base_g = floor(g * (L - S) / (n_groups - 1)) (0 for a single group), so the first window
 * starts at line 0 and the last ends at line L; *coverage = lines inside some window / L.     */
int32_t rr_make_windows(uint64_t region_bytes, uint32_t words_per_lane, uint64_t window_bytes,
                        uint32_t n_groups, uint32_t policy, uint64_t seed,
                        rr_window_t *out_host /*HOST n_groups*/, double *coverage);

/* ---- windows and work in proportion to each group's capacity (host only) ---------------------
 * Paper, Section 2.3 (each resource group run on its own): on B200 a group's throughput is capped
 * by its shared translation path whatever its SM count, so equal work per SM makes the largest
 * groups finish last.  Given an integer weight per group (its measured solo GB/s, say), with
 * P_g = w_0 + .. + w_(g-1) and T = P_G, group g gets
 *   lines [floor(L*P_g/T), floor(L*P_(g+1)/T))      (windows tile the region, uniform density)
 *   warps [floor(V*P_g/T), floor(V*P_(g+1)/T))      (V = n_warps logical warps)
 * for use with RR_MODE_POOLED.  warp_start_host receives n_groups+1 entries.  RR_ERR_RANGE if a
 * group is left without lines or warps, the weights sum above 2^32-1, or a window exceeds
 * max_window_bytes (0 = no limit; pass the measured reach).                                    */
int32_t rr_make_weighted_windows(uint64_t region_bytes, uint32_t words_per_lane, uint32_t n_groups,
                                 const uint32_t *weight_host, uint32_t n_warps,
                                 uint64_t max_window_bytes, rr_window_t *out_host,
                                 uint32_t *warp_start_host);

/* ---- plateau, cliff and reach from a size sweep (host only) --------------------------------
 * Paper, Section 2.1 / Figure 1 (throughput collapses once the region outgrows the translation
 * reach).  size_bytes strictly increasing.  plateau = lower median of GB/s over
 * 4 GiB <= size <= 32 GiB; a cliff exists iff a larger size has GB/s < 0.8 plateau; reach =
 * largest size before it with GB/s >= 0.9 plateau.  Returns 1 (cliff), 0 (none) or an error.  */
int32_t rr_reach(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                 double *plateau, uint64_t *reach_bytes);

/* Next size to measure when refining the reach (host only).  Paper, Section 2.1 / Figure 1: a
 * sweep brackets the cliff between two of its sizes.  With good = the reach rr_reach finds in
 * the sweep so far and bad = the smallest measured size above it, the next point is
 * mid = floor((good + bad) / 2 / step_bytes) * step_bytes.  Returns 1 and *next_size = mid while
 * bad - good > step_bytes and good < mid < bad; 0 (and *next_size = 0) when the refinement is
 * finished or there is no cliff; an error code as rr_reach.  The caller measures that size,
 * inserts the point and asks again: a point is judged by rr_reach alone.                      */
int32_t rr_reach_next(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                      uint64_t step_bytes, uint64_t *next_size);

/* How far one SM's own translation cache reaches (host only).  The experiment of Section 2.1
 * with one window per SM gives a rate per window size (sizes strictly increasing).  The level
 * small windows sustain is the middle one of the first three rates (the first rate if fewer);
 * *reach_bytes = the last size of the leading run of points with rate >= keep * level
 * (0 < keep <= 1); the first size if even that one falls short.                               */
int32_t rr_sm_reach(const uint64_t *size_bytes, const double *gbps, uint32_t n_points, double keep,
                    uint64_t *reach_bytes);

/* One window per SM, the SMs of a resource group side by side (host only).  Paper, Section 2.4
 * gives each group one chunk; this finer plan gives every active SM a window id of its own,
 * handed out group by group (groups in increasing number, SMs in increasing id), so that
 * windows laid out in id order put the windows of a group's SMs next to each other and each
 * group still stays inside one stretch below its reach.  group_of_sm, owner_of_sm: HOST [nsm];
 * inactive SMs stay RR_SM_INACTIVE.  *n_owners = number of ids (= active SMs).                 */
int32_t rr_owner_map(const uint16_t *group_of_sm, uint32_t nsm, uint16_t *owner_of_sm,
                     uint32_t *n_owners);

/* Size of the moving sub-windows of RR_INDEX_PHASED (host only): the slice an SM works through
 * is cut into the smallest power-of-two number of parts (at most max_parts) that makes a part
 * no larger than a quarter of the SM's reach (two phases can be live at once and should both
 * fit with room to spare); *sub_bytes = ceil(slice_bytes / *parts).                            */
int32_t rr_phase_window(uint64_t slice_bytes, uint64_t sm_reach_bytes, uint32_t max_parts,
                        uint32_t *parts, uint64_t *sub_bytes);

/* New capacity weights from one observed pooled run (host only).  Paper, Section 2.3: a group's
 * throughput belongs to the group.  Group g did work[g] units and its last SM finished
 * finish_ns[g] after the common start (0 = not seen).  In integers:
 *   rate_g = max(1, floor(work_g * 2^48 / finish_g));  unseen groups get
 *   max(1, smallest seen rate / 1024);  weight_g = max(1, floor((rate_g * scale + T/2) / T)),
 *   T = sum of rates.
 * RR_ERR_RANGE if no group finished any work.  Feed the weights to rr_make_weighted_windows,
 * run again, repeat until rr_finish_spread_ppm is small.                                       */
int32_t rr_rebalance_weights(const uint32_t *work, const uint64_t *finish_ns, uint32_t n_groups,
                             uint32_t scale, uint32_t *weight);

/* When each group finished, from the per-SM timers rr_read_block_times returns (host only):
 * the common start is the earliest start over the SMs that ran; finish_ns[g] = latest end over
 * group g's SMs that ran minus that start (at least 1; 0 if none ran); *span_ns = latest end
 * overall minus the common start.  RR_ERR_MAP if an SM that ran names a group >= n_groups.     */
int32_t rr_group_finish(const uint64_t *t_start, const uint64_t *t_end, const uint16_t *group_of_sm,
                        uint32_t nsm, uint32_t n_groups, uint64_t *finish_ns, uint64_t *span_ns);

/* (latest - earliest) / latest finish over the groups that ran, in parts per million, rounded
 * down (host only).                                                                            */
int32_t rr_finish_spread_ppm(const uint64_t *finish_ns, uint32_t n_groups, uint32_t *ppm);

/* How evenly a set of windows covers the region (host only): *covered = lines inside at least
 * one window; *depth_min / *depth_max = smallest / largest number of windows over a covered
 * line.  With equal work and equal sizes the read density at a line is proportional to its
 * depth, so depth_max / depth_min says how uniform overlapping windows (policy 2) are.         */
int32_t rr_window_cover(const rr_window_t *windows, uint32_t n_groups, uint64_t n_lines,
                        uint64_t *covered, uint32_t *depth_min, uint32_t *depth_max);

#ifdef __cplusplus
}
#endif
#endif /* RR_H_ */
