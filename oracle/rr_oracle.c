/*
 * rr_oracle.c -- plain CPU definition of the random-line-read path.
 *
 * TEST INFRASTRUCTURE.  Only the tests, the smoke check and the CPU-baseline leg
 * of the benchmark may call this file.  It shares no source, header, table or
 * constant generator with the CUDA library; the product never falls back to it.
 *
 * What it defines (the paper gives prose only, so every definition below is a
 * stated reading of that prose):
 *   - Section 2.1 (the basic benchmark): each warp fetches whole lines of 32 words
 *     (32-, 64- or 128-bit) at random positions inside a memory region; here the region has
 *     known contents (a hash of the word index), the random line comes from a
 *     counter-based generator, and what is read is folded into two checksums per
 *     warp so that a reader can prove which lines were touched.
 *   - Section 2.1, second experiment and Section 2.4: all warps of an SM (of an SM
 *     group) are held to one chunk (window) of the region.
 *   - Section 2.2: the SM x SM pair-throughput matrix is rearranged into groups;
 *     here: average-linkage agglomeration with a largest-gap cut.
 *
 * Everything is written as the definition, one word at a time, with no blocking,
 * fusion or reordering.  The only parallelism is an OpenMP loop over warps (or over
 * the words of a fill), which are independent by definition.
 *
 * Pins (see tests/test_oracle_*.py): the public SplitMix64 output streams, a
 * big-integer brute force over tiny materialised buffers, window invariants,
 * the width identity, a sequential mode that must fold the whole buffer, draw
 * statistics, and planted partitions for the clustering.
 * Parity unpinned: orc_reach() thresholds (0.8 / 0.9 of the plateau) are a
 * reading with no external truth; only their bookkeeping is tested.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_RANGE (-3)
#define ORC_ERR_MAP (-4)

#define ORC_INDEX_RANDOM 0u
#define ORC_INDEX_STRIDE 1u
#define ORC_SM_INACTIVE 0xFFFFu

/* ---- O1: mixing function and buffer contents --------------------------------
 * sm64(x) is the first output of a SplitMix64 generator whose state is x:
 * add the golden-ratio increment, then the three-step finaliser.              */
static const uint64_t ORC_GAMMA = 0x9E3779B97F4A7C15ULL;

uint64_t orc_sm64(uint64_t x)
{
    uint64_t z = x + ORC_GAMMA;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* Contents of 32-bit word i of the buffer (i counts from the buffer start). */
uint32_t orc_word(uint64_t i)
{
    return (uint32_t)(orc_sm64(i) & 0xFFFFFFFFULL);
}

void orc_fill(uint32_t *dst, uint64_t first_word, uint64_t n_words)
{
    int64_t n = (int64_t)n_words;
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k)
        dst[k] = orc_word(first_word + (uint64_t)k);
}

/* ---- O2: line index ----------------------------------------------------------
 * A keyed, random-access SplitMix64 stream per logical warp v:
 *   k_seed = sm64(seed);  k_v = sm64(k_seed ^ v);  r(seed,v,i) = sm64(k_v + i*gamma)
 * i.e. the i-th output (0-based) of a SplitMix64 generator with state k_v.      */
uint64_t orc_warp_key(uint64_t seed, uint64_t v)
{
    return orc_sm64(orc_sm64(seed) ^ v);
}

uint64_t orc_draw(uint64_t seed, uint64_t v, uint64_t i)
{
    return orc_sm64(orc_warp_key(seed, v) + i * ORC_GAMMA);
}

/* Line (in units of 128*W bytes from the buffer start) read i of warp v hits.
 * RANDOM: base + (r mod n).  STRIDE (sequential control, Section 2.1 last
 * paragraph): base + ((i * n_warps_total + v) mod n).                          */
uint64_t orc_line(uint32_t index_mode, uint64_t seed, uint64_t v, uint64_t n_warps_total,
                  uint64_t i, uint64_t base, uint64_t n)
{
    uint64_t idx;
    if (index_mode == ORC_INDEX_STRIDE)
        idx = (i * n_warps_total + v) % n;
    else
        idx = orc_draw(seed, v, i) % n;
    return base + idx;
}

/* ---- O3: what one warp reads and folds ---------------------------------------
 * Lane l of the warp reads W consecutive 32-bit words starting at word
 * line*32W + l*W; every 32-bit word is folded separately:
 *   X = xor of all words, S = sum of all words mod 2^32,
 * over 32 lanes, W words, R reads (a line drawn twice counts twice).            */
void orc_warp_checksum(uint32_t index_mode, uint64_t seed, uint64_t v, uint64_t n_warps_total,
                       uint64_t first_read, uint64_t reads, uint32_t W,
                       uint64_t base, uint64_t n, uint32_t *X, uint32_t *S)
{
    uint32_t x = 0, s = 0;
    for (uint64_t t = 0; t < reads; ++t) {
        uint64_t line = orc_line(index_mode, seed, v, n_warps_total, first_read + t, base, n);
        for (uint32_t lane = 0; lane < 32; ++lane) {
            for (uint32_t w = 0; w < W; ++w) {
                uint64_t j = line * 32u * W + (uint64_t)lane * W + w;
                uint32_t word = orc_word(j);
                x ^= word;
                s += word;
            }
        }
    }
    *X = x;
    *S = s;
}

/* ---- O3b: windows that move with time ------------------------------------------
 * Section 1.3 wants each warp confined to a part of memory smaller than the reach; the
 * paper fixes that part for good.  Reading for hardware whose per-SM translation
 * cache is smaller than its share of memory: the warp's window of n lines is cut into
 * Q = ceil(n / sub_lines) sub-windows [floor(n q / Q), floor(n (q+1) / Q)); reads come
 * in phases of phase_reads reads, phase p = floor(i / phase_reads) of a warp's stream
 * (i = absolute read counter) draws uniformly inside sub-window p mod Q.  Over Q
 * phases every line of the window is equally likely; at any moment a warp is held to
 * n/Q lines.  With sub_lines >= n this is the plain random mode.
 * stagger shifts the cycle: sub-window (p + stagger) mod Q.  In per-SM mode SM s of nsm
 * uses stagger = floor(s * Q / nsm), so that SMs sharing one window (all of memory, say)
 * are spread over its sub-windows instead of crowding into one.                      */
uint64_t orc_line_phased(uint64_t seed, uint64_t v, uint64_t i, uint64_t base, uint64_t n,
                         uint64_t phase_reads, uint64_t sub_lines, uint64_t stagger)
{
    uint64_t Q = (n + sub_lines - 1) / sub_lines;
    uint64_t q = (i / phase_reads + stagger) % Q;
    uint64_t lo = n * q / Q, hi = n * (q + 1) / Q; /* n < 2^32, Q <= n: fits 64 bits */
    return base + lo + orc_draw(seed, v, i) % (hi - lo);
}

void orc_warp_checksum_phased(uint64_t seed, uint64_t v, uint64_t first_read, uint64_t reads,
                              uint32_t W, uint64_t base, uint64_t n, uint64_t phase_reads,
                              uint64_t sub_lines, uint64_t stagger, uint32_t *X, uint32_t *S)
{
    uint32_t x = 0, s = 0;
    for (uint64_t t = 0; t < reads; ++t) {
        uint64_t line = orc_line_phased(seed, v, first_read + t, base, n, phase_reads, sub_lines,
                                        stagger);
        for (uint32_t lane = 0; lane < 32; ++lane)
            for (uint32_t w = 0; w < W; ++w) {
                uint32_t word = orc_word(line * 32u * W + (uint64_t)lane * W + w);
                x ^= word;
                s += word;
            }
    }
    *X = x;
    *S = s;
}

static int orc_width_ok(uint32_t W) { return W == 1 || W == 2 || W == 4; }

/* ---- O3c: a stream that mixes sequential and random reads ----------------------------
 * Section 2.1 ends by noting that sequential access runs faster than random access; a real
 * workload is often a blend.  Reading: with a period k >= 1, read i of a warp's stream is
 * sequential when i mod k == 0 -- it is read number i/k of the warp's sequential walk,
 * line = base + ((i/k) * n_warps_total + v) mod n, exactly the STRIDE rule applied to the
 * counter i/k -- and random otherwise (the RANDOM rule at the same i).  k = 1 is the
 * sequential mode; as k grows the stream tends to the random mode.                     */
uint64_t orc_line_mixed(uint64_t seed, uint64_t v, uint64_t n_warps_total, uint64_t i,
                        uint64_t base, uint64_t n, uint64_t mix_period)
{
    if (i % mix_period == 0)
        return orc_line(ORC_INDEX_STRIDE, seed, v, n_warps_total, i / mix_period, base, n);
    return orc_line(ORC_INDEX_RANDOM, seed, v, n_warps_total, i, base, n);
}

void orc_warp_checksum_mixed(uint64_t seed, uint64_t v, uint64_t n_warps_total, uint64_t first_read,
                             uint64_t reads, uint32_t W, uint64_t base, uint64_t n,
                             uint64_t mix_period, uint32_t *X, uint32_t *S)
{
    uint32_t x = 0, s = 0;
    for (uint64_t t = 0; t < reads; ++t) {
        uint64_t line = orc_line_mixed(seed, v, n_warps_total, first_read + t, base, n, mix_period);
        for (uint32_t lane = 0; lane < 32; ++lane)
            for (uint32_t w = 0; w < W; ++w) {
                uint32_t word = orc_word(line * 32u * W + (uint64_t)lane * W + w);
                x ^= word;
                s += word;
            }
    }
    *X = x;
    *S = s;
}

/* Per-SM mode with the mixed stream; arguments as orc_read_per_sm.                      */
int32_t orc_read_per_sm_mixed(uint64_t region_bytes, uint32_t W, uint32_t nsm, uint32_t wps,
                              uint64_t first_read, uint64_t reads, uint64_t seed,
                              const uint16_t *group_of_sm, const uint32_t *win_base,
                              const uint32_t *win_n, uint32_t n_groups, uint64_t mix_period,
                              uint32_t *out)
{
    if (!orc_width_ok(W) || !out || nsm == 0 || wps == 0 || mix_period == 0) return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    if (group_of_sm) {
        if (!win_base || !win_n || n_groups == 0) return ORC_ERR_ARG;
        for (uint32_t g = 0; g < n_groups; ++g)
            if (win_n[g] == 0 || (uint64_t)win_base[g] + win_n[g] > L) return ORC_ERR_RANGE;
        for (uint32_t s = 0; s < nsm; ++s)
            if (group_of_sm[s] != ORC_SM_INACTIVE && group_of_sm[s] >= n_groups) return ORC_ERR_MAP;
    }
    uint64_t total = (uint64_t)nsm * wps;
    int64_t nw = (int64_t)total;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t v = 0; v < nw; ++v) {
        uint32_t sm = (uint32_t)(v / wps);
        uint64_t base = 0, n = L;
        if (group_of_sm) {
            if (group_of_sm[sm] == ORC_SM_INACTIVE) {
                out[2 * v] = 0;
                out[2 * v + 1] = 0;
                continue;
            }
            base = win_base[group_of_sm[sm]];
            n = win_n[group_of_sm[sm]];
        }
        orc_warp_checksum_mixed(seed, (uint64_t)v, total, first_read, reads, W, base, n, mix_period,
                                &out[2 * v], &out[2 * v + 1]);
    }
    return ORC_OK;
}

/* Per-SM mode with moving windows (see orc_line_phased); arguments as orc_read_per_sm.
 * nsm = 0 with group_of_sm = NULL is not accepted; for logical warps over the whole
 * region pass one group covering everything.                                        */
int32_t orc_read_per_sm_phased(uint64_t region_bytes, uint32_t W, uint32_t nsm, uint32_t wps,
                               uint64_t first_read, uint64_t reads, uint64_t seed,
                               const uint16_t *group_of_sm, const uint32_t *win_base,
                               const uint32_t *win_n, uint32_t n_groups, uint64_t phase_reads,
                               uint64_t phase_window_bytes, uint32_t *out)
{
    if (!orc_width_ok(W) || !out || nsm == 0 || wps == 0 || phase_reads == 0) return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    uint64_t sub = phase_window_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull || sub == 0) return ORC_ERR_RANGE;
    if (group_of_sm) {
        if (!win_base || !win_n || n_groups == 0) return ORC_ERR_ARG;
        for (uint32_t g = 0; g < n_groups; ++g)
            if (win_n[g] == 0 || (uint64_t)win_base[g] + win_n[g] > L) return ORC_ERR_RANGE;
        for (uint32_t s = 0; s < nsm; ++s)
            if (group_of_sm[s] != ORC_SM_INACTIVE && group_of_sm[s] >= n_groups) return ORC_ERR_MAP;
    }
    int64_t nw = (int64_t)nsm * wps;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t v = 0; v < nw; ++v) {
        uint32_t sm = (uint32_t)(v / wps);
        uint64_t base = 0, n = L;
        if (group_of_sm) {
            if (group_of_sm[sm] == ORC_SM_INACTIVE) {
                out[2 * v] = 0;
                out[2 * v + 1] = 0;
                continue;
            }
            base = win_base[group_of_sm[sm]];
            n = win_n[group_of_sm[sm]];
        }
        uint64_t Q = (n + sub - 1) / sub;
        uint64_t stagger = (uint64_t)sm * Q / nsm;
        orc_warp_checksum_phased(seed, (uint64_t)v, first_read, reads, W, base, n, phase_reads, sub,
                                 stagger, &out[2 * v], &out[2 * v + 1]);
    }
    return ORC_OK;
}

/* The same logical-mode read performed on a real buffer in host memory (filled with
 * orc_fill): the line is indexed literally instead of regenerated.  This is the CPU
 * analogue of the method for sizes that fit host RAM, and a second statement of what a
 * "coalesced line read" touches.  buf holds region_bytes/4 words.                     */
int32_t orc_read_logical_materialised(const uint32_t *buf, uint64_t region_bytes, uint32_t W,
                                      uint64_t n_warps, uint64_t first_read, uint64_t reads,
                                      uint64_t seed, uint32_t *out)
{
    if (!buf || !out || !orc_width_ok(W)) return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    int64_t nw = (int64_t)n_warps;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t v = 0; v < nw; ++v) {
        uint32_t x = 0, s = 0;
        for (uint64_t t = 0; t < reads; ++t) {
            uint64_t line = orc_draw(seed, (uint64_t)v, first_read + t) % L;
            const uint32_t *p = buf + line * 32u * W; /* the 32*W words of that line */
            for (uint32_t k = 0; k < 32u * W; ++k) {
                x ^= p[k];
                s += p[k];
            }
        }
        out[2 * v] = x;
        out[2 * v + 1] = s;
    }
    return ORC_OK;
}

/* Logical-warp mode: v = 0 .. n_warps-1, window = the whole region.
 * out holds n_warps pairs {X, S}.                                               */
int32_t orc_read_logical(uint64_t region_bytes, uint32_t W, uint32_t index_mode,
                         uint64_t n_warps, uint64_t first_read, uint64_t reads,
                         uint64_t seed, uint32_t *out)
{
    if (!orc_width_ok(W) || index_mode > 1 || !out) return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    int64_t nw = (int64_t)n_warps;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t v = 0; v < nw; ++v)
        orc_warp_checksum(index_mode, seed, (uint64_t)v, n_warps, first_read, reads, W, 0, L,
                          &out[2 * v], &out[2 * v + 1]);
    return ORC_OK;
}

/* Logical-warp mode with a window per warp: warp v reads inside window v mod n_windows.
 * Section 2.1 tries the simplest restriction first -- every SM on its own random half --
 * and finds no benefit; this is the same control one level finer, a window chosen per
 * warp with no regard for SMs or groups (windows from orc_make_windows policy 1).       */
int32_t orc_read_logical_windows(uint64_t region_bytes, uint32_t W, uint64_t n_warps,
                                 uint64_t first_read, uint64_t reads, uint64_t seed,
                                 const uint32_t *win_base, const uint32_t *win_n,
                                 uint32_t n_windows, uint32_t *out)
{
    if (!orc_width_ok(W) || !out || !win_base || !win_n || n_windows == 0) return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    for (uint32_t g = 0; g < n_windows; ++g)
        if (win_n[g] == 0 || (uint64_t)win_base[g] + win_n[g] > L) return ORC_ERR_RANGE;
    int64_t nw = (int64_t)n_warps;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t v = 0; v < nw; ++v) {
        uint32_t g = (uint32_t)((uint64_t)v % n_windows);
        orc_warp_checksum(ORC_INDEX_RANDOM, seed, (uint64_t)v, n_warps, first_read, reads, W,
                          win_base[g], win_n[g], &out[2 * v], &out[2 * v + 1]);
    }
    return ORC_OK;
}

/* Per-SM mode: v = smid*wps + warp; window = windows[group_of_sm[smid]] (whole
 * region when group_of_sm is NULL); inactive SMs (0xFFFF) give {0,0}.
 * out holds nsm*wps pairs.                                                      */
int32_t orc_read_per_sm(uint64_t region_bytes, uint32_t W, uint32_t index_mode,
                        uint32_t nsm, uint32_t wps, uint64_t first_read, uint64_t reads,
                        uint64_t seed, const uint16_t *group_of_sm,
                        const uint32_t *win_base, const uint32_t *win_n, uint32_t n_groups,
                        uint32_t *out)
{
    if (!orc_width_ok(W) || index_mode > 1 || !out || nsm == 0 || wps == 0) return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    if (group_of_sm) {
        if (!win_base || !win_n || n_groups == 0) return ORC_ERR_ARG;
        for (uint32_t g = 0; g < n_groups; ++g)
            if (win_n[g] == 0 || (uint64_t)win_base[g] + win_n[g] > L) return ORC_ERR_RANGE;
        for (uint32_t s = 0; s < nsm; ++s)
            if (group_of_sm[s] != ORC_SM_INACTIVE && group_of_sm[s] >= n_groups) return ORC_ERR_MAP;
    }
    uint64_t total = (uint64_t)nsm * wps;
    int64_t nw = (int64_t)total;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t v = 0; v < nw; ++v) {
        uint32_t sm = (uint32_t)(v / wps);
        uint64_t base = 0, n = L;
        if (group_of_sm) {
            if (group_of_sm[sm] == ORC_SM_INACTIVE) {
                out[2 * v] = 0;
                out[2 * v + 1] = 0;
                continue;
            }
            base = win_base[group_of_sm[sm]];
            n = win_n[group_of_sm[sm]];
        }
        orc_warp_checksum(index_mode, seed, (uint64_t)v, total, first_read, reads, W, base, n,
                          &out[2 * v], &out[2 * v + 1]);
    }
    return ORC_OK;
}

/* ---- O4: windows (Section 1.3: a window below the reach, half the memory as the simple
 * case; Section 2.4) ---------------------------------------------------------------
 * L lines are cut into K = ceil(L / S_lines) chunks of floor(L/K) lines, the last
 * one running to L.  policy 0: group g takes chunk g mod K.  policy 1 (the
 * paper's naive control, one "group" per SM): chunk sm64(seed ^ g) mod K.
 * coverage = distinct chunks used / K.
 * policy 2 (Section 1.3 only asks that each warp's window stay below the reach; the
 * windows need not be disjoint): G windows of exactly S_lines lines, evenly spaced with
 * overlap, base_g = floor(g * (L - S_lines) / (G - 1)) (base 0 when G = 1), so the first
 * starts at line 0 and the last ends at line L.  coverage = lines inside at least one
 * window / L, which is 1 exactly when no step between bases exceeds S_lines.           */
int32_t orc_make_windows(uint64_t region_bytes, uint32_t W, uint64_t window_bytes,
                         uint32_t n_groups, uint32_t policy, uint64_t seed,
                         uint32_t *win_base, uint32_t *win_n, double *coverage)
{
    if (!orc_width_ok(W) || n_groups == 0 || policy > 2 || !win_base || !win_n) return ORC_ERR_ARG;
    uint64_t line_bytes = 128ull * W;
    uint64_t L = region_bytes / line_bytes;
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    uint64_t S = window_bytes / line_bytes;
    if (S < 1) S = 1;
    if (S > L) S = L;
    if (policy == 2) {
        uint64_t covered = 0, end_prev = 0;
        for (uint32_t g = 0; g < n_groups; ++g) {
            uint64_t base = n_groups > 1 ? (uint64_t)g * (L - S) / (n_groups - 1) : 0;
            win_base[g] = (uint32_t)base;
            win_n[g] = (uint32_t)S;
            /* bases do not decrease: lines newly covered by this window */
            uint64_t from = base > end_prev ? base : end_prev;
            if (base + S > from) covered += base + S - from;
            if (base + S > end_prev) end_prev = base + S;
        }
        if (coverage) *coverage = (double)covered / (double)L;
        return ORC_OK;
    }
    uint64_t K = (L + S - 1) / S;
    uint64_t chunk = L / K;
    unsigned char *used = (unsigned char *)calloc((size_t)K, 1);
    if (!used) return ORC_ERR_ARG;
    for (uint32_t g = 0; g < n_groups; ++g) {
        uint64_t c = (policy == 1) ? (orc_sm64(seed ^ (uint64_t)g) % K) : ((uint64_t)g % K);
        uint64_t lo = c * chunk;
        uint64_t hi = (c == K - 1) ? L : (c + 1) * chunk;
        win_base[g] = (uint32_t)lo;
        win_n[g] = (uint32_t)(hi - lo);
        used[c] = 1;
    }
    uint64_t distinct = 0;
    for (uint64_t c = 0; c < K; ++c) distinct += used[c];
    free(used);
    if (coverage) *coverage = (double)distinct / (double)K;
    return ORC_OK;
}

/* How evenly a set of windows covers the region: for every line, depth = number of
 * windows that contain it.  With equal work per window and equal window sizes the read
 * density at a line is proportional to its depth.  Returns the number of lines with
 * depth >= 1 and the smallest and largest depth over those lines (plain sweep over the
 * 2G window edges).                                                                   */
int32_t orc_window_cover(const uint32_t *win_base, const uint32_t *win_n, uint32_t n_groups,
                         uint64_t n_lines, uint64_t *covered, uint32_t *depth_min,
                         uint32_t *depth_max)
{
    if (!win_base || !win_n || !covered || !depth_min || !depth_max || n_groups == 0)
        return ORC_ERR_ARG;
    for (uint32_t g = 0; g < n_groups; ++g)
        if (win_n[g] == 0 || (uint64_t)win_base[g] + win_n[g] > n_lines) return ORC_ERR_RANGE;
    uint64_t *edge = (uint64_t *)malloc(sizeof(uint64_t) * 2 * n_groups);
    if (!edge) return ORC_ERR_ARG;
    for (uint32_t g = 0; g < n_groups; ++g) {
        edge[2 * g] = win_base[g];
        edge[2 * g + 1] = (uint64_t)win_base[g] + win_n[g];
    }
    /* insertion sort of the distinct edge positions: G <= a few hundred */
    uint32_t ne = 2 * n_groups;
    for (uint32_t i = 1; i < ne; ++i) {
        uint64_t x = edge[i];
        uint32_t j = i;
        while (j > 0 && edge[j - 1] > x) {
            edge[j] = edge[j - 1];
            --j;
        }
        edge[j] = x;
    }
    uint64_t cov = 0;
    uint32_t dmin = 0xFFFFFFFFu, dmax = 0;
    for (uint32_t i = 0; i + 1 < ne; ++i) {
        uint64_t a = edge[i], b = edge[i + 1];
        if (b == a) continue;
        uint32_t depth = 0; /* windows containing the stretch [a, b) */
        for (uint32_t g = 0; g < n_groups; ++g)
            if (win_base[g] <= a && b <= (uint64_t)win_base[g] + win_n[g]) ++depth;
        if (depth == 0) continue;
        cov += b - a;
        if (depth < dmin) dmin = depth;
        if (depth > dmax) dmax = depth;
    }
    free(edge);
    *covered = cov;
    *depth_min = dmin == 0xFFFFFFFFu ? 0 : dmin;
    *depth_max = dmax;
    return ORC_OK;
}

/* ---- O4b: windows and work in proportion to each group's capacity ----------------
 * Section 2.3 runs every resource group on its own and finds that a group's throughput
 * is a property of the group.  If every SM does the same work, the groups with the most
 * SMs per unit of capacity finish last and set the time.  Reading: give group g the
 * integer weight w_g (its measured solo throughput); with P_g = w_0 + .. + w_(g-1) and
 * T = P_G, group g owns
 *   lines  [floor(L * P_g / T), floor(L * P_(g+1) / T))   -- windows tile the region
 *   warps  [floor(V * P_g / T), floor(V * P_(g+1) / T))   -- logical warps, same rule
 * so reads stay uniformly dense over the region and each group's share of the work
 * matches its share of the capacity.  warp_start receives G+1 entries.
 * Errors: a group left without lines or without warps, or a window above max_window_bytes
 * (0 = no limit).                                                                  */
int32_t orc_make_weighted_windows(uint64_t region_bytes, uint32_t W, uint32_t n_groups,
                                  const uint32_t *weight, uint64_t n_warps,
                                  uint64_t max_window_bytes, uint32_t *win_base,
                                  uint32_t *win_n, uint32_t *warp_start)
{
    if (!orc_width_ok(W) || n_groups == 0 || !weight || !win_base || !win_n || !warp_start ||
        n_warps == 0 || n_warps > 0xFFFFFFFFull)
        return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    uint64_t T = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        if (weight[g] == 0) return ORC_ERR_ARG;
        T += weight[g];
    }
    if (T > 0xFFFFFFFFull) return ORC_ERR_RANGE; /* keeps L*P and V*P inside 64 bits */
    uint64_t P = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        uint64_t lo = L * P / T, hi = L * (P + weight[g]) / T;
        uint64_t vlo = n_warps * P / T, vhi = n_warps * (P + weight[g]) / T;
        if (hi == lo || vhi == vlo) return ORC_ERR_RANGE;
        if (max_window_bytes && (hi - lo) * 128ull * W > max_window_bytes) return ORC_ERR_RANGE;
        win_base[g] = (uint32_t)lo;
        win_n[g] = (uint32_t)(hi - lo);
        warp_start[g] = (uint32_t)vlo;
        P += weight[g];
    }
    warp_start[n_groups] = (uint32_t)n_warps;
    return ORC_OK;
}

/* Pooled mode: logical warps v = 0 .. V-1 (V = warp_start[G]); warp v belongs to the group
 * g with warp_start[g] <= v < warp_start[g+1] and reads inside that group's window.
 * Which SM performs which of its reads is left to the machine; the checksums do not
 * depend on it.  out holds V pairs {X, S}.                                          */
int32_t orc_read_pooled(uint64_t region_bytes, uint32_t W, uint32_t n_groups,
                        const uint32_t *win_base, const uint32_t *win_n,
                        const uint32_t *warp_start, uint64_t first_read, uint64_t reads,
                        uint64_t seed, uint32_t *out)
{
    if (!orc_width_ok(W) || n_groups == 0 || !win_base || !win_n || !warp_start || !out)
        return ORC_ERR_ARG;
    uint64_t L = region_bytes / (128ull * W);
    if (L == 0 || L > 0xFFFFFFFFull) return ORC_ERR_RANGE;
    if (warp_start[0] != 0) return ORC_ERR_ARG;
    for (uint32_t g = 0; g < n_groups; ++g) {
        if (warp_start[g + 1] < warp_start[g]) return ORC_ERR_ARG;
        if (win_n[g] == 0 || (uint64_t)win_base[g] + win_n[g] > L) return ORC_ERR_RANGE;
    }
    uint64_t V = warp_start[n_groups];
    int64_t nw = (int64_t)V;
    /* one loop over all warps (they are independent), so that every host core has work
     * whatever the number of groups; the owner of warp v is looked up by its range */
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t v = 0; v < nw; ++v) {
        uint32_t g = 0;
        while (!((uint64_t)v >= warp_start[g] && (uint64_t)v < warp_start[g + 1])) ++g;
        orc_warp_checksum(ORC_INDEX_RANDOM, seed, (uint64_t)v, V, first_read, reads, W,
                          win_base[g], win_n[g], &out[2 * v], &out[2 * v + 1]);
    }
    return ORC_OK;
}

/* ---- O5: SM x SM matrix -> groups (Section 2.2, Figures 2 and 3) ---------------
 * 1. symmetrise off-diagonal entries in double: t = (T_ij + T_ji) / 2; with flag
 *    ORC_CLUSTER_SOLO_NORMALISE, divide by the two SMs' solo rates on the diagonal:
 *    t = t / (T_ii + T_jj), so that an SM that is slower on its own is not mistaken
 *    for a contended one (1.0 = the pair runs as fast as the two solos together)
 * 2. quantise: q = rint(t * 2^20 / lower-median(t)), clamped to 2^32-1
 * 3. average linkage on q (small q = contended = close): exact integer pair sums,
 *    means compared by cross-multiplication, ties -> smallest (a,b); a cluster is
 *    named by its smallest member; height of a merge = sum / (na*nb) in double
 * 4. cut: apply the first k merges, k chosen among cuts leaving 2..floor(n/3)
 *    clusters to maximise h[k] - h[k-1]; the first maximum wins
 * 5. null rule: sigma = 1.4826 * MAD of the q of pairs in different clusters after
 *    the cut, divided by sqrt of the number of pairs averaged in merge k (so it
 *    is the noise of the height that defines the gap); gap < 4 sigma, or gap below
 *    1 % of the median pair rate (a faint background pattern) -> one group
 * 6. labels: groups numbered by their smallest SM id
 * heights (optional) receives the n-1 merge heights.                            */
static int cmp_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}
static int cmp_u32(const void *a, const void *b)
{
    uint32_t x = *(const uint32_t *)a, y = *(const uint32_t *)b;
    return (x > y) - (x < y);
}

#define ORC_CLUSTER_SOLO_NORMALISE 1u

int32_t orc_cluster(const float *T, uint32_t n, uint32_t flags, int32_t *group_of_sm,
                    uint32_t *n_groups, double *confidence, double *heights)
{
    if (!T || !group_of_sm || !n_groups || n < 2 || n > 256 || flags > 1) return ORC_ERR_ARG;
    size_t m = (size_t)n * (n - 1) / 2;
    double *t = (double *)malloc(sizeof(double) * (size_t)n * n);
    double *sorted = (double *)malloc(sizeof(double) * m);
    uint32_t *q = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)n * n);
    uint64_t *sum = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)n * n);
    uint32_t *size = (uint32_t *)malloc(sizeof(uint32_t) * n);
    uint32_t *alive = (uint32_t *)malloc(sizeof(uint32_t) * n);
    uint32_t *merge_a = (uint32_t *)malloc(sizeof(uint32_t) * n);
    uint32_t *merge_b = (uint32_t *)malloc(sizeof(uint32_t) * n);
    uint64_t *merge_pairs = (uint64_t *)malloc(sizeof(uint64_t) * n);
    double *h = (double *)malloc(sizeof(double) * n);
    uint32_t *between = (uint32_t *)malloc(sizeof(uint32_t) * (m ? m : 1));
    int32_t rc = ORC_OK;
    if (!t || !sorted || !q || !sum || !size || !alive || !merge_a || !merge_b || !merge_pairs ||
        !h || !between) {
        rc = ORC_ERR_ARG;
        goto done;
    }

    /* 1. symmetrise, validate */
    {
        size_t k = 0;
        for (uint32_t i = 0; i < n; ++i)
            for (uint32_t j = i + 1; j < n; ++j) {
                double a = (double)T[(size_t)i * n + j], b = (double)T[(size_t)j * n + i];
                if (!(a > 0.0) || !(b > 0.0) || isinf(a) || isinf(b)) {
                    rc = ORC_ERR_ARG;
                    goto done;
                }
                double s = (a + b) * 0.5;
                if (flags & ORC_CLUSTER_SOLO_NORMALISE) {
                    double di = (double)T[(size_t)i * n + i], dj = (double)T[(size_t)j * n + j];
                    if (!(di > 0.0) || !(dj > 0.0) || isinf(di) || isinf(dj)) {
                        rc = ORC_ERR_ARG;
                        goto done;
                    }
                    s = s / (di + dj);
                }
                t[(size_t)i * n + j] = s;
                t[(size_t)j * n + i] = s;
                sorted[k++] = s;
            }
    }
    /* 2. quantise against the lower median */
    qsort(sorted, m, sizeof(double), cmp_double);
    {
        double med = sorted[(m - 1) / 2];
        for (uint32_t i = 0; i < n; ++i)
            for (uint32_t j = 0; j < n; ++j) {
                if (i == j) {
                    q[(size_t)i * n + j] = 0;
                    continue;
                }
                double r = rint(t[(size_t)i * n + j] * 1048576.0 / med);
                q[(size_t)i * n + j] = (r >= 4294967295.0) ? 0xFFFFFFFFu : (uint32_t)r;
            }
    }
    /* 3. average linkage */
    for (uint32_t i = 0; i < n; ++i) {
        size[i] = 1;
        alive[i] = 1;
        for (uint32_t j = 0; j < n; ++j) sum[(size_t)i * n + j] = q[(size_t)i * n + j];
    }
    for (uint32_t step = 0; step + 1 < n; ++step) {
        int have = 0;
        uint32_t ba = 0, bb = 0;
        uint64_t bs = 0, bp = 1;
        for (uint32_t a = 0; a < n; ++a) {
            if (!alive[a]) continue;
            for (uint32_t b = a + 1; b < n; ++b) {
                if (!alive[b]) continue;
                uint64_t s = sum[(size_t)a * n + b];
                uint64_t p = (uint64_t)size[a] * size[b];
                /* s/p < bs/bp  <=>  s*bp < bs*p  (all < 2^60 for n <= 256) */
                if (!have || s * bp < bs * p) {
                    have = 1;
                    ba = a;
                    bb = b;
                    bs = s;
                    bp = p;
                }
            }
        }
        merge_a[step] = ba;
        merge_b[step] = bb;
        merge_pairs[step] = bp;
        h[step] = (double)bs / (double)bp;
        for (uint32_t c = 0; c < n; ++c) {
            if (!alive[c] || c == ba || c == bb) continue;
            uint64_t s = sum[(size_t)ba * n + c] + sum[(size_t)bb * n + c];
            sum[(size_t)ba * n + c] = s;
            sum[(size_t)c * n + ba] = s;
        }
        size[ba] += size[bb];
        alive[bb] = 0;
    }
    if (heights)
        for (uint32_t k = 0; k + 1 < n; ++k) heights[k] = h[k];

    /* 4. cut */
    for (uint32_t i = 0; i < n; ++i) group_of_sm[i] = 0;
    *n_groups = 1;
    if (confidence) *confidence = 0.0;
    {
        uint32_t max_clusters = n / 3;
        if (max_clusters < 2) goto done; /* too few SMs for a group level */
        uint32_t k_lo = n - max_clusters, k_hi = n - 2, best_k = 0;
        double best_gap = -1.0;
        for (uint32_t k = k_lo; k <= k_hi; ++k) {
            double gap = h[k] - h[k - 1];
            if (gap > best_gap) {
                best_gap = gap;
                best_k = k;
            }
        }
        /* replay the first best_k merges; parent[] by smallest member */
        uint32_t *rep = alive; /* reuse: representative of each SM */
        for (uint32_t i = 0; i < n; ++i) rep[i] = i;
        for (uint32_t k = 0; k < best_k; ++k)
            for (uint32_t i = 0; i < n; ++i)
                if (rep[i] == merge_b[k]) rep[i] = merge_a[k];
        /* 5. null rule */
        size_t nb = 0;
        for (uint32_t i = 0; i < n; ++i)
            for (uint32_t j = i + 1; j < n; ++j)
                if (rep[i] != rep[j]) between[nb++] = q[(size_t)i * n + j];
        qsort(between, nb, sizeof(uint32_t), cmp_u32);
        uint32_t bmed = between[(nb - 1) / 2];
        for (size_t k = 0; k < nb; ++k)
            between[k] = between[k] > bmed ? between[k] - bmed : bmed - between[k];
        qsort(between, nb, sizeof(uint32_t), cmp_u32);
        double mad = (double)between[(nb - 1) / 2];
        double sigma = (1.4826 * mad) / sqrt((double)merge_pairs[best_k]);
        double conf = sigma > 0.0 ? best_gap / sigma : (best_gap > 0.0 ? INFINITY : 0.0);
        if (confidence) *confidence = conf;
        /* Section 2.2 sets the fainter background structure of its matrix aside:
         * a gap below 1 % of the median pair rate (2^20 in these units) is no group boundary */
        if (!(best_gap >= 4.0 * sigma) || !(best_gap >= 10485.76)) goto done; /* one group */
        /* 6. canonical labels: representatives are smallest members */
        uint32_t G = 0;
        for (uint32_t i = 0; i < n; ++i)
            if (rep[i] == i) merge_pairs[i] = G++; /* reuse as label-of-representative */
        for (uint32_t i = 0; i < n; ++i) group_of_sm[i] = (int32_t)merge_pairs[rep[i]];
        *n_groups = G;
    }
done:
    free(t);
    free(sorted);
    free(q);
    free(sum);
    free(size);
    free(alive);
    free(merge_a);
    free(merge_b);
    free(merge_pairs);
    free(h);
    free(between);
    return rc;
}

/* ---- O6: plateau, cliff, reach from a (size, GB/s) sweep (Section 2.1, Fig. 1) ---
 * plateau = median GB/s over 4 GiB <= N <= 32 GiB (upper of the two middle values
 * is NOT averaged: lower median); a cliff exists iff some larger N has GB/s below
 * 0.8 plateau; reach = largest N with GB/s >= 0.9 plateau below the first such N.
 * Returns 1 and *reach_bytes if a cliff exists, 0 if absent.                     */
int32_t orc_reach(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                  double *plateau, uint64_t *reach_bytes)
{
    if (!size_bytes || !gbps || n_points == 0 || !plateau || !reach_bytes) return ORC_ERR_ARG;
    double *mid = (double *)malloc(sizeof(double) * n_points);
    if (!mid) return ORC_ERR_ARG;
    uint32_t nm = 0;
    const uint64_t GiB = 1ull << 30;
    for (uint32_t k = 0; k < n_points; ++k) {
        if (k && size_bytes[k] <= size_bytes[k - 1]) {
            free(mid);
            return ORC_ERR_ARG; /* sizes must increase */
        }
        if (size_bytes[k] >= 4 * GiB && size_bytes[k] <= 32 * GiB) mid[nm++] = gbps[k];
    }
    if (nm == 0) {
        free(mid);
        return ORC_ERR_RANGE;
    }
    qsort(mid, nm, sizeof(double), cmp_double);
    double P = mid[(nm - 1) / 2];
    free(mid);
    *plateau = P;
    *reach_bytes = 0;
    int32_t cliff = 0;
    uint32_t first_bad = n_points;
    for (uint32_t k = 0; k < n_points; ++k)
        if (size_bytes[k] > 32 * GiB && gbps[k] < 0.8 * P) {
            cliff = 1;
            first_bad = k;
            break;
        }
    for (uint32_t k = 0; k < first_bad; ++k)
        if (gbps[k] >= 0.9 * P) *reach_bytes = size_bytes[k];
    return cliff;
}

/* ---- O6b: next size to measure when refining the reach ---------------------------
 * The sweep of Section 2.1 / Fig. 1 only brackets the cliff between two of its sizes.
 * Reading: bisect between the reach found so far (good) and the smallest measured size
 * above it (bad) on a grid of `step` bytes: mid = floor((good + bad) / 2 / step) * step.
 * Returns 1 and *next_size = mid while bad - good > step and good < mid < bad; 0 when
 * the refinement is finished or the sweep shows no cliff.  A measured point is judged by
 * orc_reach itself (it is appended to the sweep and the rule is applied again), so there
 * is no second acceptance threshold.                                                 */
int32_t orc_reach_next(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                       uint64_t step_bytes, uint64_t *next_size)
{
    if (!next_size || step_bytes == 0) return ORC_ERR_ARG;
    double plateau;
    uint64_t good;
    int32_t rc = orc_reach(size_bytes, gbps, n_points, &plateau, &good);
    if (rc < 0) return rc;
    *next_size = 0;
    if (rc == 0) return 0;
    uint64_t bad = 0;
    for (uint32_t k = 0; k < n_points; ++k)
        if (size_bytes[k] > good) {
            bad = size_bytes[k];
            break; /* sizes increase: the first one above is the smallest */
        }
    if (bad == 0 || bad - good <= step_bytes) return 0;
    uint64_t mid = (good + bad) / 2 / step_bytes * step_bytes;
    if (mid <= good || mid >= bad) return 0;
    *next_size = mid;
    return 1;
}

/* ---- O7: how far one SM's own translation cache reaches ------------------------------
 * Same experiment as Section 2.1 with one window per SM: rate versus window size, sizes
 * increasing.  Reading: the level the small windows sustain is the middle one of the
 * first three rates (the only rate if fewer than three points); the reach is the last
 * size of the leading run of points whose rate is at least keep * that level.  A sweep
 * whose very first point already falls short returns its first size.                  */
int32_t orc_sm_reach(const uint64_t *size_bytes, const double *gbps, uint32_t n_points,
                     double keep, uint64_t *reach_bytes)
{
    if (!size_bytes || !gbps || !reach_bytes || n_points == 0 || !(keep > 0.0) || keep > 1.0)
        return ORC_ERR_ARG;
    for (uint32_t k = 1; k < n_points; ++k)
        if (size_bytes[k] <= size_bytes[k - 1]) return ORC_ERR_ARG;
    double top;
    if (n_points >= 3) {
        double a = gbps[0], b = gbps[1], c = gbps[2];
        /* middle of three */
        if ((a <= b && b <= c) || (c <= b && b <= a)) top = b;
        else if ((b <= a && a <= c) || (c <= a && a <= b)) top = a;
        else top = c;
    } else {
        top = gbps[0];
    }
    *reach_bytes = size_bytes[0];
    for (uint32_t k = 0; k < n_points; ++k) {
        if (gbps[k] >= keep * top) *reach_bytes = size_bytes[k];
        else break;
    }
    return ORC_OK;
}

/* ---- O8: one window per SM, the SMs of a resource group side by side -----------------
 * Section 2.4 gives every group one chunk.  A finer reading that still keeps every group
 * below its reach: every active SM gets a window id of its own, ids handed out group by
 * group (groups in increasing number, SMs of a group in increasing SM id), so that with
 * windows laid out in id order the windows of one group's SMs are neighbours and together
 * form the group's chunk.  Inactive SMs (0xFFFF) stay inactive.  Returns the number of ids. */
int32_t orc_owner_map(const uint16_t *group_of_sm, uint32_t nsm, uint16_t *owner_of_sm,
                      uint32_t *n_owners)
{
    if (!group_of_sm || !owner_of_sm || !n_owners || nsm == 0 || nsm > 65535u) return ORC_ERR_ARG;
    uint32_t next = 0;
    uint32_t max_g = 0;
    int any = 0;
    for (uint32_t s = 0; s < nsm; ++s)
        if (group_of_sm[s] != ORC_SM_INACTIVE) {
            if (!any || group_of_sm[s] > max_g) max_g = group_of_sm[s];
            any = 1;
        }
    for (uint32_t s = 0; s < nsm; ++s) owner_of_sm[s] = ORC_SM_INACTIVE;
    if (any)
        for (uint32_t g = 0; g <= max_g; ++g)
            for (uint32_t s = 0; s < nsm; ++s)
                if (group_of_sm[s] == g) owner_of_sm[s] = (uint16_t)next++;
    *n_owners = next;
    return ORC_OK;
}

/* ---- O9: size of the moving sub-windows (see orc_line_phased) ---------------------------
 * Two phases of a warp's stream can be live at once, and the SM's translation cache
 * should hold both with room to spare: the slice an SM works through is cut into the
 * smallest power-of-two number of parts (at most max_parts) that makes a part no larger
 * than a quarter of the SM's reach; sub = ceil(slice / parts).                        */
int32_t orc_phase_window(uint64_t slice_bytes, uint64_t sm_reach_bytes, uint32_t max_parts,
                         uint32_t *parts, uint64_t *sub_bytes)
{
    if (!parts || !sub_bytes || slice_bytes == 0 || sm_reach_bytes == 0 || max_parts == 0)
        return ORC_ERR_ARG;
    uint32_t q = 1;
    /* slice / q > reach / 4   <=>   4 * slice > reach * q   (exact in integers) */
    while (q < max_parts && (unsigned __int128)4 * slice_bytes > (unsigned __int128)sm_reach_bytes * q)
        q *= 2;
    *parts = q;
    *sub_bytes = (slice_bytes + q - 1) / q;
    return ORC_OK;
}

/* ---- O10: new capacity weights from one observed run -----------------------------------
 * Section 2.3: a group's throughput belongs to the group.  After a run in which group g
 * did work[g] units and its last SM finished finish_ns[g] after the common start, the
 * group has shown the rate work/finish.  Reading, in integers so that nothing depends on
 * rounding mode: rate_g = max(1, floor(work_g * 2^48 / finish_g)); a group that was not
 * seen (finish 0 or no work) keeps a token rate of max(1, smallest seen rate / 1024); the
 * new weight is the rate's share of `scale`, rounded half up, at least 1:
 *   w_g = max(1, floor((rate_g * scale + total / 2) / total)),  total = sum of rates.
 * At a fixed point (every group finishing together) the weights reproduce the work
 * shares.  (work < 2^32, scale < 2^32: every product stays below 2^128.)              */
int32_t orc_rebalance_weights(const uint32_t *work, const uint64_t *finish_ns, uint32_t n_groups,
                              uint32_t scale, uint32_t *weight)
{
    typedef unsigned __int128 u128;
    if (!work || !finish_ns || !weight || n_groups == 0 || scale == 0) return ORC_ERR_ARG;
    u128 *rate = (u128 *)malloc(sizeof(u128) * n_groups);
    if (!rate) return ORC_ERR_ARG;
    u128 slowest = 0;
    int seen = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        rate[g] = 0;
        if (finish_ns[g] == 0 || work[g] == 0) continue;
        rate[g] = ((u128)work[g] << 48) / finish_ns[g];
        if (rate[g] == 0) rate[g] = 1;
        if (!seen || rate[g] < slowest) slowest = rate[g];
        seen = 1;
    }
    if (!seen) {
        free(rate);
        return ORC_ERR_RANGE; /* no group finished any work */
    }
    u128 token = slowest / 1024;
    if (token == 0) token = 1;
    u128 total = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        if (rate[g] == 0) rate[g] = token;
        total += rate[g];
    }
    for (uint32_t g = 0; g < n_groups; ++g) {
        u128 w = (rate[g] * scale + total / 2) / total;
        weight[g] = w == 0 ? 1u : (uint32_t)w;
    }
    free(rate);
    return ORC_OK;
}

/* When each group finished, from the per-SM block timers of one run (ns; t_end = 0 for an
 * SM that ran no block): the common start is the earliest start over the SMs that ran,
 * finish[g] = latest end over group g's SMs that ran, minus that start (at least 1; 0 if
 * none of the group's SMs ran); *span = latest end overall minus the common start.    */
int32_t orc_group_finish(const uint64_t *t_start, const uint64_t *t_end, const uint16_t *group_of_sm,
                         uint32_t nsm, uint32_t n_groups, uint64_t *finish_ns, uint64_t *span_ns)
{
    if (!t_start || !t_end || !group_of_sm || !finish_ns || !span_ns || nsm == 0 || n_groups == 0)
        return ORC_ERR_ARG;
    uint64_t begin = 0, last = 0;
    int any = 0;
    for (uint32_t s = 0; s < nsm; ++s) {
        if (t_end[s] == 0) continue;
        if (!any || t_start[s] < begin) begin = t_start[s];
        if (!any || t_end[s] > last) last = t_end[s];
        any = 1;
    }
    for (uint32_t g = 0; g < n_groups; ++g) finish_ns[g] = 0;
    *span_ns = any ? last - begin : 0;
    for (uint32_t s = 0; s < nsm; ++s) {
        if (t_end[s] == 0 || group_of_sm[s] == ORC_SM_INACTIVE) continue;
        if (group_of_sm[s] >= n_groups) return ORC_ERR_MAP;
        uint64_t f = t_end[s] > begin ? t_end[s] - begin : 1;
        if (f > finish_ns[group_of_sm[s]]) finish_ns[group_of_sm[s]] = f;
    }
    return ORC_OK;
}

/* (latest - earliest) / latest over the groups that ran, in parts per million, rounded
 * down: how far from finishing together the groups of a balanced run were.            */
int32_t orc_finish_spread_ppm(const uint64_t *finish_ns, uint32_t n_groups, uint32_t *ppm)
{
    if (!finish_ns || !ppm || n_groups == 0) return ORC_ERR_ARG;
    uint64_t lo = 0, hi = 0;
    int seen = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        if (finish_ns[g] == 0) continue;
        if (!seen || finish_ns[g] < lo) lo = finish_ns[g];
        if (!seen || finish_ns[g] > hi) hi = finish_ns[g];
        seen = 1;
    }
    *ppm = seen ? (uint32_t)(((unsigned __int128)(hi - lo) * 1000000u) / hi) : 0u;
    return ORC_OK;
}

/* ---- O11: rate and overlap of one two-SM probe (Section 2.2, Fig. 2) --------------------
 * Each chosen SM performs total_reads / 2 line reads of 128 bytes (the part whose checksums
 * are verified) and then keeps reading until the other SM has finished its own share, so
 * that two SMs of different speed still run side by side for the whole measurement;
 * extra_lines[i] counts what SM i read beyond its share.  The pair's throughput counts every
 * line read by both SMs over the union of their two intervals,
 *   GB/s = bytes / (latest end - earliest start)        (timers in ns, so bytes/ns = GB/s)
 * and the figure only means contention if the two ran side by side:
 *   overlap = (earliest end - latest start) / (latest end - earliest start), 0 if disjoint.
 * A solo run (one SM) has overlap 1 and no extra lines.  An SM that claimed nothing or never
 * ended: -6.                                                                            */
#define ORC_ERR_SM_UNCOVERED (-6)
int32_t orc_probe_rate(const uint64_t *t_start, const uint64_t *t_end, const uint32_t *claim,
                       const uint64_t *extra_lines, uint32_t solo, uint64_t total_reads,
                       double *gbps, double *seconds, double *overlap)
{
    if (!t_start || !t_end || !claim || !extra_lines || !gbps || !seconds || !overlap || solo > 1)
        return ORC_ERR_ARG;
    uint32_t k = solo ? 1 : 2;
    for (uint32_t i = 0; i < k; ++i)
        if (claim[i] == 0 || t_end[i] == 0 || t_end[i] < t_start[i]) return ORC_ERR_SM_UNCOVERED;
    uint64_t s_lo = t_start[0], s_hi = t_start[0], e_lo = t_end[0], e_hi = t_end[0];
    uint64_t lines = total_reads / 2 + extra_lines[0];
    if (k == 2) {
        if (t_start[1] < s_lo) s_lo = t_start[1];
        if (t_start[1] > s_hi) s_hi = t_start[1];
        if (t_end[1] < e_lo) e_lo = t_end[1];
        if (t_end[1] > e_hi) e_hi = t_end[1];
        lines += total_reads / 2 + extra_lines[1];
    }
    uint64_t span = e_hi - s_lo;
    uint64_t bytes = lines * 128ull;
    *seconds = (double)span * 1e-9;
    *gbps = span ? (double)bytes / (double)span : 0.0;
    *overlap = (span && e_lo > s_hi) ? (double)(e_lo - s_hi) / (double)span : 0.0;
    return ORC_OK;
}
