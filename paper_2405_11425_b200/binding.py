"""ctypes binding of librr.so: the same entry points as include/rr.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; nothing here computes.  Device
buffers are passed as torch tensors (or raw integer addresses); host tables as numpy arrays.
Importing this module fails loudly if the library has not been built -- there is no fallback.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from pathlib import Path

import numpy as np

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "librr.so"

RR_OK = 0
RR_ERR_ARG, RR_ERR_ALIGN, RR_ERR_RANGE, RR_ERR_MAP, RR_ERR_CUDA = -1, -2, -3, -4, -5
RR_ERR_SM_UNCOVERED, RR_ERR_TIMEOUT, RR_ERR_CHECK, RR_ERR_UNSUPPORTED = -6, -7, -8, -9
RR_ERR_STATIC_LIMIT = -10
RR_STATIC_MAX_SM, RR_STATIC_SCRATCH_BYTES = 192, 5888
RR_MAX_SM, RR_MAX_GROUPS, RR_MAX_WARPS_PER_SM, RR_SM_INACTIVE = 256, 256, 32, 0xFFFF
RR_MODE_LOGICAL, RR_MODE_PER_SM, RR_MODE_POOLED = 0, 1, 2
RR_INDEX_RANDOM, RR_INDEX_STRIDE, RR_INDEX_PHASED, RR_INDEX_MIXED = 0, 1, 2, 3
RR_VARIANT_LDG, RR_VARIANT_LDG_CHECKED, RR_VARIANT_PACKED = 0, 1, 2
RR_VARIANT_SORTED = 3

EXPORTS = (
    "rr_strerror", "rr_last_cuda_error", "rr_device_info", "rr_scratch_bytes", "rr_fill",
    "rr_random_read", "rr_read_report", "rr_probe_pair", "rr_probe_matrix_scratch_bytes",
    "rr_probe_matrix", "rr_cluster", "rr_make_windows", "rr_reach", "rr_random_read_static",
    "rr_gpc_map", "rr_make_weighted_windows",
    "rr_read_block_times", "rr_host_counters", "rr_probe_rate", "rr_reach_next", "rr_sm_reach",
    "rr_owner_map", "rr_phase_window", "rr_rebalance_weights", "rr_finish_spread_ppm",
    "rr_window_cover", "rr_group_finish", "rr_probe_rows",
)


class RRError(RuntimeError):
    def __init__(self, code: int, where: str):
        lib = _load()
        msg = lib.rr_strerror(code).decode()
        if code == RR_ERR_CUDA or code == RR_ERR_UNSUPPORTED:
            msg += ": " + lib.rr_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({code})")
        self.code = code


class _Window(ctypes.Structure):
    _fields_ = [("base_line", ctypes.c_uint32), ("n_lines", ctypes.c_uint32)]


class _ReadParams(ctypes.Structure):
    _fields_ = [
        ("buf", ctypes.c_void_p), ("region_bytes", ctypes.c_uint64),
        ("words_per_lane", ctypes.c_uint32), ("mode", ctypes.c_uint32),
        ("index_mode", ctypes.c_uint32), ("n_warps", ctypes.c_uint32),
        ("warps_per_sm", ctypes.c_uint32), ("nsm", ctypes.c_uint32),
        ("reads_per_warp", ctypes.c_uint64), ("first_read", ctypes.c_uint64),
        ("seed", ctypes.c_uint64), ("group_of_sm", ctypes.c_void_p),
        ("windows", ctypes.c_void_p), ("n_groups", ctypes.c_uint32),
        ("variant", ctypes.c_uint32), ("unroll", ctypes.c_uint32),
        ("pool_block_reads", ctypes.c_uint32), ("warp_start", ctypes.c_void_p),
        ("phase_reads", ctypes.c_uint32), ("mix_period", ctypes.c_uint32),
        ("phase_window_bytes", ctypes.c_uint64),
        ("sort_parts", ctypes.c_uint32), ("sort_reads", ctypes.c_uint32),
    ]


class _Result(ctypes.Structure):
    _fields_ = [
        ("seconds_event", ctypes.c_double), ("seconds_device", ctypes.c_double),
        ("bytes", ctypes.c_uint64), ("gbps", ctypes.c_double), ("status", ctypes.c_uint32),
        ("violations", ctypes.c_uint32), ("sms_covered", ctypes.c_uint32),
        ("blocks_run", ctypes.c_uint32),
    ]


class _DeviceInfo(ctypes.Structure):
    _fields_ = [
        ("nsm_prop", ctypes.c_uint32), ("nsm_reg", ctypes.c_uint32),
        ("cc_major", ctypes.c_uint32), ("cc_minor", ctypes.c_uint32),
        ("free_bytes", ctypes.c_uint64), ("total_bytes", ctypes.c_uint64),
        ("mem_clock_khz", ctypes.c_uint32), ("bus_width_bits", ctypes.c_uint32),
        ("l2_bytes", ctypes.c_uint64), ("smem_per_sm", ctypes.c_uint32),
        ("smem_per_block_optin", ctypes.c_uint32), ("theoretical_gbps", ctypes.c_double),
        ("name", ctypes.c_char * 64), ("uuid", ctypes.c_char * 40),
    ]


@dataclass
class ReadResult:
    seconds_event: float
    seconds_device: float
    bytes: int
    gbps: float
    status: int
    violations: int
    sms_covered: int
    blocks_run: int


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2405_11425_b200.build` "
            "(nvcc, sm_100a).  There is no CPU fallback.")
    lib = ctypes.CDLL(str(LIB_PATH))
    for name in EXPORTS:
        if not hasattr(lib, name):
            raise ImportError(f"{LIB_PATH} does not export {name}")
    u64, u32, i32, p, d = (ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int32, ctypes.c_void_p,
                           ctypes.c_double)
    lib.rr_strerror.restype = ctypes.c_char_p
    lib.rr_strerror.argtypes = [i32]
    lib.rr_last_cuda_error.restype = ctypes.c_char_p
    lib.rr_last_cuda_error.argtypes = []
    lib.rr_device_info.restype = i32
    lib.rr_device_info.argtypes = [p, p, p]
    lib.rr_scratch_bytes.restype = ctypes.c_size_t
    lib.rr_scratch_bytes.argtypes = []
    lib.rr_fill.restype = i32
    lib.rr_fill.argtypes = [p, u64, p]
    lib.rr_random_read.restype = i32
    lib.rr_random_read.argtypes = [p, p, p, p, p]
    lib.rr_random_read_static.restype = i32
    lib.rr_random_read_static.argtypes = [p, p, p, p]
    lib.rr_read_block_times.restype = i32
    lib.rr_read_block_times.argtypes = [p, u32, p, p, p]
    lib.rr_read_report.restype = i32
    lib.rr_read_report.argtypes = [p, p, p, p]
    lib.rr_probe_pair.restype = i32
    lib.rr_probe_pair.argtypes = [p, u64, u32, u32, u64, u32, u64, p, p, p, p]
    lib.rr_probe_matrix_scratch_bytes.restype = ctypes.c_size_t
    lib.rr_probe_matrix_scratch_bytes.argtypes = [u32]
    lib.rr_probe_matrix.restype = i32
    lib.rr_probe_matrix.argtypes = [p, u64, u64, u32, u64, u32, p, u32, p, p, p, p, p]
    lib.rr_probe_rows.restype = i32
    lib.rr_probe_rows.argtypes = [p, u64, u64, u32, u64, u32, u32, u32, p, u32, p, p, p, p, p]
    lib.rr_probe_rate.restype = i32
    lib.rr_probe_rate.argtypes = [p, p, p, p, u32, u64, p, p, p]
    lib.rr_reach_next.restype = i32
    lib.rr_reach_next.argtypes = [p, p, u32, u64, p]
    lib.rr_sm_reach.restype = i32
    lib.rr_sm_reach.argtypes = [p, p, u32, d, p]
    lib.rr_owner_map.restype = i32
    lib.rr_owner_map.argtypes = [p, u32, p, p]
    lib.rr_phase_window.restype = i32
    lib.rr_phase_window.argtypes = [u64, u64, u32, p, p]
    lib.rr_rebalance_weights.restype = i32
    lib.rr_rebalance_weights.argtypes = [p, p, u32, u32, p]
    lib.rr_group_finish.restype = i32
    lib.rr_group_finish.argtypes = [p, p, p, u32, u32, p, p]
    lib.rr_finish_spread_ppm.restype = i32
    lib.rr_finish_spread_ppm.argtypes = [p, u32, p]
    lib.rr_window_cover.restype = i32
    lib.rr_window_cover.argtypes = [p, u32, u64, p, p, p]
    lib.rr_cluster.restype = i32
    lib.rr_cluster.argtypes = [p, u32, u32, p, p, p, p, p, p]
    lib.rr_gpc_map.restype = i32
    lib.rr_gpc_map.argtypes = [p, p, p, u32, p]
    lib.rr_make_windows.restype = i32
    lib.rr_make_windows.argtypes = [u64, u32, u64, u32, u32, u64, p, p]
    lib.rr_make_weighted_windows.restype = i32
    lib.rr_make_weighted_windows.argtypes = [u64, u32, u32, p, u32, u64, p, p]
    lib.rr_reach.restype = i32
    lib.rr_reach.argtypes = [p, p, u32, p, p]
    lib.rr_host_counters.restype = i32
    lib.rr_host_counters.argtypes = [p]
    _lib = lib
    return lib


def _dev(x) -> int:
    """Device address of a torch tensor (or a raw integer address)."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    return int(x.data_ptr())


def _stream(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def _check(rc: int, where: str):
    if rc != RR_OK:
        raise RRError(rc, where)


def rr_strerror(code: int) -> str:
    return _load().rr_strerror(code).decode()


def rr_device_info(scratch=None, stream=None) -> dict:
    """Facts of the current device; nsm_reg (%nsmid) is read only when a scratch buffer is given."""
    info = _DeviceInfo()
    _check(_load().rr_device_info(ctypes.byref(info), _dev(scratch),
                                  _stream(stream) if scratch is not None else None),
           "rr_device_info")
    out = {k: getattr(info, k) for k, _ in _DeviceInfo._fields_}
    out["name"] = info.name.decode()
    out["uuid"] = info.uuid.decode()
    return out


def rr_host_counters() -> dict:
    """How often the library really asked the runtime for occupancy, attributes, events, facts."""
    c = (ctypes.c_uint64 * 4)()
    _check(_load().rr_host_counters(c), "rr_host_counters")
    return dict(zip(("occupancy_queries", "attribute_sets", "event_creates",
                     "device_fact_queries"), (int(x) for x in c)))


def rr_scratch_bytes() -> int:
    return int(_load().rr_scratch_bytes())


def rr_probe_matrix_scratch_bytes(nsm: int) -> int:
    return int(_load().rr_probe_matrix_scratch_bytes(nsm))


def rr_fill(buf, n_words: int, stream=None) -> None:
    _check(_load().rr_fill(_dev(buf), n_words, _stream(stream)), "rr_fill")


class ReadParams:
    """Host-side copy of rr_read_params_t; keeps the numpy tables it points to alive."""

    def __init__(self, buf, region_bytes: int, *, W: int = 1, mode: int = RR_MODE_PER_SM,
                 index_mode: int = RR_INDEX_RANDOM, n_warps: int = 0, warps_per_sm: int = 32,
                 nsm: int = 0, reads_per_warp: int = 0, first_read: int = 0, seed: int = 0,
                 group_of_sm=None, windows=None, variant: int = RR_VARIANT_LDG, unroll: int = 0,
                 warp_start=None, pool_block_reads: int = 0, phase_reads: int = 0,
                 phase_window_bytes: int = 0, mix_period: int = 0, sort_parts: int = 0,
                 sort_reads: int = 0):
        self._groups = None
        self._windows = None
        self._warp_start = None
        if warp_start is not None:
            self._warp_start = np.ascontiguousarray(warp_start, dtype=np.uint32)
        n_groups = 0
        if group_of_sm is not None:
            self._groups = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
            nsm = nsm or int(self._groups.shape[0])
        if windows is not None:
            self._windows = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
            n_groups = int(self._windows.shape[0])
        self.c = _ReadParams(
            _dev(buf), region_bytes, W, mode, index_mode, n_warps, warps_per_sm, nsm,
            reads_per_warp, first_read, seed,
            self._groups.ctypes.data if self._groups is not None else None,
            self._windows.ctypes.data if self._windows is not None else None,
            n_groups, variant, unroll, pool_block_reads,
            self._warp_start.ctypes.data if self._warp_start is not None else None,
            phase_reads, mix_period, phase_window_bytes, sort_parts, sort_reads)


def _result(r: _Result) -> ReadResult:
    return ReadResult(r.seconds_event, r.seconds_device, int(r.bytes), r.gbps, r.status,
                      r.violations, r.sms_covered, r.blocks_run)


def rr_random_read(params: ReadParams, out, scratch, *, timed: bool = True, stream=None):
    """Launches the read; `timed` = synchronous with a ReadResult, else asynchronous (None)."""
    res = _Result()
    rc = _load().rr_random_read(ctypes.byref(params.c), _dev(out), _dev(scratch),
                                ctypes.byref(res) if timed else None, _stream(stream))
    _check(rc, "rr_random_read")
    return _result(res) if timed else None


def rr_random_read_static(params: ReadParams, out, *, report: bool = True, stream=None):
    """rr_random_read for callers that cannot allocate: the scratch is built into the library.

    `report` = wait and return a ReadResult (device-side timing only), else queue and return
    None.  Calls on one device share the built-in scratch and must not overlap."""
    res = _Result()
    rc = _load().rr_random_read_static(ctypes.byref(params.c), _dev(out),
                                       ctypes.byref(res) if report else None, _stream(stream))
    _check(rc, "rr_random_read_static")
    return _result(res) if report else None


def rr_read_report(params: ReadParams, scratch, stream=None) -> ReadResult:
    res = _Result()
    _check(_load().rr_read_report(ctypes.byref(params.c), _dev(scratch), ctypes.byref(res),
                                  _stream(stream)), "rr_read_report")
    return _result(res)


def rr_read_block_times(scratch, nsm: int, stream=None):
    """(t_start, t_end) uint64[nsm] in ns of every SM's block in the last read on this scratch."""
    t0 = np.zeros(nsm, dtype=np.uint64)
    t1 = np.zeros(nsm, dtype=np.uint64)
    _check(_load().rr_read_block_times(_dev(scratch), nsm, t0.ctypes.data, t1.ctypes.data,
                                       _stream(stream)), "rr_read_block_times")
    return t0, t1


def rr_probe_pair(buf, region_bytes: int, sm_a: int, sm_b: int, total_reads: int,
                  warps_per_sm: int, seed: int, out, scratch, stream=None) -> ReadResult:
    res = _Result()
    _check(_load().rr_probe_pair(_dev(buf), region_bytes, sm_a, sm_b, total_reads, warps_per_sm,
                                 seed, _dev(out), _dev(scratch), ctypes.byref(res),
                                 _stream(stream)), "rr_probe_pair")
    return _result(res)


class _ProbeStats(ctypes.Structure):
    _fields_ = [("overlap_min", ctypes.c_double), ("pairs_below_goal", ctypes.c_uint32),
                ("reruns", ctypes.c_uint32), ("relaunched", ctypes.c_uint32)]


def rr_probe_matrix(buf, region_bytes: int, total_reads: int, warps_per_sm: int, seed: int,
                    repeats: int, nsm: int, out, scratch, stream=None, *, with_overlaps=False):
    """Returns (T float32[nsm,nsm], stats dict) -- plus the per-pair overlap matrix if asked."""
    T = np.zeros((nsm, nsm), dtype=np.float32)
    ov = np.ones((nsm, nsm), dtype=np.float32) if with_overlaps else None
    st = _ProbeStats()
    _check(_load().rr_probe_matrix(_dev(buf), region_bytes, total_reads, warps_per_sm, seed,
                                   repeats, T.ctypes.data, nsm, _dev(out), _dev(scratch),
                                   ctypes.byref(st), ov.ctypes.data if with_overlaps else None,
                                   _stream(stream)), "rr_probe_matrix")
    stats = {"overlap_min": float(st.overlap_min), "pairs_below_goal": int(st.pairs_below_goal),
             "reruns": int(st.reruns), "relaunched": int(st.relaunched)}
    return (T, stats, ov) if with_overlaps else (T, stats)


def rr_probe_rows(buf, region_bytes: int, total_reads: int, warps_per_sm: int, seed: int,
                  repeats: int, row_begin: int, row_end: int, T, out, scratch, overlaps=None,
                  stream=None) -> dict:
    """Probes rows [row_begin, row_end) into the caller's matrix T (float32 [nsm, nsm], updated
    in place; `overlaps` likewise if given).  Returns the stats of these rows."""
    if T.dtype != np.float32 or T.ndim != 2 or T.shape[0] != T.shape[1] or \
            not T.flags["C_CONTIGUOUS"]:
        raise RRError(RR_ERR_ARG, "rr_probe_rows")
    st = _ProbeStats()
    _check(_load().rr_probe_rows(_dev(buf), region_bytes, total_reads, warps_per_sm, seed, repeats,
                                 row_begin, row_end, T.ctypes.data, T.shape[0], _dev(out),
                                 _dev(scratch), ctypes.byref(st),
                                 overlaps.ctypes.data if overlaps is not None else None,
                                 _stream(stream)), "rr_probe_rows")
    return {"overlap_min": float(st.overlap_min), "pairs_below_goal": int(st.pairs_below_goal),
            "reruns": int(st.reruns), "relaunched": int(st.relaunched)}


def rr_probe_rate(t_start, t_end, claim, solo: bool, total_reads: int, extra_lines=(0, 0)):
    """(GB/s, seconds, overlap) of one probe from its timers (host rule, no GPU involved)."""
    a = np.ascontiguousarray(t_start, dtype=np.uint64)
    b = np.ascontiguousarray(t_end, dtype=np.uint64)
    c = np.ascontiguousarray(claim, dtype=np.uint32)
    x = np.ascontiguousarray(extra_lines, dtype=np.uint64)
    g, sec, ov = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    _check(_load().rr_probe_rate(a.ctypes.data, b.ctypes.data, c.ctypes.data, x.ctypes.data,
                                 1 if solo else 0, total_reads, ctypes.byref(g), ctypes.byref(sec),
                                 ctypes.byref(ov)), "rr_probe_rate")
    return float(g.value), float(sec.value), float(ov.value)


RR_CLUSTER_SOLO_NORMALISE = 1


def rr_cluster(T, scratch, flags: int = 0, stream=None):
    """Returns (group_of_sm int32[n], n_groups, confidence, heights float64[n-1])."""
    T = np.ascontiguousarray(T, dtype=np.float32)
    n = int(T.shape[0])
    if T.ndim != 2 or T.shape[1] != n:
        raise RRError(RR_ERR_ARG, "rr_cluster")
    groups = np.zeros(n, dtype=np.int32)
    heights = np.zeros(max(n - 1, 1), dtype=np.float64)
    ng = ctypes.c_uint32()
    conf = ctypes.c_double()
    _check(_load().rr_cluster(T.ctypes.data, n, flags, _dev(scratch), groups.ctypes.data,
                              ctypes.byref(ng), ctypes.byref(conf), heights.ctypes.data,
                              _stream(stream)), "rr_cluster")
    return groups, int(ng.value), float(conf.value), heights[: n - 1]


def rr_gpc_map(scratch, nsm: int, stream=None):
    """Returns (gpc_of_sm int32[nsm], n_gpcs) from thread-block-cluster placement."""
    g = np.zeros(nsm, dtype=np.int32)
    ng = ctypes.c_uint32()
    _check(_load().rr_gpc_map(_dev(scratch), g.ctypes.data, ctypes.byref(ng), nsm,
                              _stream(stream)), "rr_gpc_map")
    return g, int(ng.value)


def rr_make_windows(region_bytes: int, W: int, window_bytes: int, n_groups: int, policy: int = 0,
                    seed: int = 0):
    """Returns ((n_groups, 2) uint32 {base_line, n_lines}, coverage)."""
    out = np.zeros((max(n_groups, 1), 2), dtype=np.uint32)
    cov = ctypes.c_double()
    _check(_load().rr_make_windows(region_bytes, W, window_bytes, n_groups, policy, seed,
                                   out.ctypes.data, ctypes.byref(cov)), "rr_make_windows")
    return out[:n_groups], float(cov.value)


def rr_make_weighted_windows(region_bytes: int, W: int, weights, n_warps: int,
                             max_window_bytes: int = 0):
    """Returns ((G, 2) uint32 windows, warp_start uint32[G+1]) in proportion to integer weights."""
    w = np.ascontiguousarray(weights, dtype=np.uint32)
    G = int(w.shape[0])
    win = np.zeros((max(G, 1), 2), dtype=np.uint32)
    ws = np.zeros(G + 1, dtype=np.uint32)
    _check(_load().rr_make_weighted_windows(region_bytes, W, G, w.ctypes.data, n_warps,
                                            max_window_bytes, win.ctypes.data, ws.ctypes.data),
           "rr_make_weighted_windows")
    return win[:G], ws


def rr_reach(size_bytes, gbps):
    """Returns (cliff_exists, plateau GB/s, reach bytes)."""
    s = np.ascontiguousarray(size_bytes, dtype=np.uint64)
    g = np.ascontiguousarray(gbps, dtype=np.float64)
    if s.shape != g.shape or s.ndim != 1:
        raise RRError(RR_ERR_ARG, "rr_reach")
    plateau = ctypes.c_double()
    r = ctypes.c_uint64()
    rc = _load().rr_reach(s.ctypes.data, g.ctypes.data, len(s), ctypes.byref(plateau),
                          ctypes.byref(r))
    if rc < 0:
        raise RRError(rc, "rr_reach")
    return bool(rc), float(plateau.value), int(r.value)


def rr_reach_next(size_bytes, gbps, step_bytes: int) -> int:
    """Next size to measure while refining the reach, or 0 when the refinement is finished."""
    s = np.ascontiguousarray(size_bytes, dtype=np.uint64)
    g = np.ascontiguousarray(gbps, dtype=np.float64)
    if s.shape != g.shape or s.ndim != 1:
        raise RRError(RR_ERR_ARG, "rr_reach_next")
    nxt = ctypes.c_uint64()
    rc = _load().rr_reach_next(s.ctypes.data, g.ctypes.data, len(s), step_bytes, ctypes.byref(nxt))
    if rc < 0:
        raise RRError(rc, "rr_reach_next")
    return int(nxt.value) if rc else 0


def rr_sm_reach(size_bytes, gbps, keep: float = 0.97) -> int:
    s = np.ascontiguousarray(size_bytes, dtype=np.uint64)
    g = np.ascontiguousarray(gbps, dtype=np.float64)
    if s.shape != g.shape or s.ndim != 1:
        raise RRError(RR_ERR_ARG, "rr_sm_reach")
    r = ctypes.c_uint64()
    _check(_load().rr_sm_reach(s.ctypes.data, g.ctypes.data, len(s), keep, ctypes.byref(r)),
           "rr_sm_reach")
    return int(r.value)


def rr_owner_map(group_of_sm):
    """(owner_of_sm uint16[nsm], n_owners): one window id per active SM, group by group."""
    g = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
    out = np.zeros(g.shape[0], dtype=np.uint16)
    n = ctypes.c_uint32()
    _check(_load().rr_owner_map(g.ctypes.data, g.shape[0], out.ctypes.data, ctypes.byref(n)),
           "rr_owner_map")
    return out, int(n.value)


def rr_phase_window(slice_bytes: int, sm_reach_bytes: int, max_parts: int = 64):
    """(parts, sub_bytes) of the moving sub-windows."""
    parts = ctypes.c_uint32()
    sub = ctypes.c_uint64()
    _check(_load().rr_phase_window(slice_bytes, sm_reach_bytes, max_parts, ctypes.byref(parts),
                                   ctypes.byref(sub)), "rr_phase_window")
    return int(parts.value), int(sub.value)


def rr_rebalance_weights(work, finish_ns, scale: int = 1_000_000) -> np.ndarray:
    w = np.ascontiguousarray(work, dtype=np.uint32)
    f = np.ascontiguousarray(finish_ns, dtype=np.uint64)
    if w.shape != f.shape or w.ndim != 1:
        raise RRError(RR_ERR_ARG, "rr_rebalance_weights")
    out = np.zeros(w.shape[0], dtype=np.uint32)
    _check(_load().rr_rebalance_weights(w.ctypes.data, f.ctypes.data, w.shape[0], scale,
                                        out.ctypes.data), "rr_rebalance_weights")
    return out


def rr_group_finish(t_start, t_end, group_of_sm, n_groups: int):
    """(finish_ns uint64[n_groups], span_ns) from the per-SM block timers of one run."""
    a = np.ascontiguousarray(t_start, dtype=np.uint64)
    b = np.ascontiguousarray(t_end, dtype=np.uint64)
    g = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
    if not (a.shape == b.shape == g.shape) or a.ndim != 1:
        raise RRError(RR_ERR_ARG, "rr_group_finish")
    out = np.zeros(n_groups, dtype=np.uint64)
    span = ctypes.c_uint64()
    _check(_load().rr_group_finish(a.ctypes.data, b.ctypes.data, g.ctypes.data, g.shape[0],
                                   n_groups, out.ctypes.data, ctypes.byref(span)),
           "rr_group_finish")
    return out, int(span.value)


def rr_finish_spread_ppm(finish_ns) -> int:
    f = np.ascontiguousarray(finish_ns, dtype=np.uint64)
    ppm = ctypes.c_uint32()
    _check(_load().rr_finish_spread_ppm(f.ctypes.data, f.shape[0], ctypes.byref(ppm)),
           "rr_finish_spread_ppm")
    return int(ppm.value)


def rr_window_cover(windows, n_lines: int):
    """(covered lines, smallest depth, largest depth) of a set of windows."""
    w = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
    cov = ctypes.c_uint64()
    lo, hi = ctypes.c_uint32(), ctypes.c_uint32()
    _check(_load().rr_window_cover(w.ctypes.data, w.shape[0], n_lines, ctypes.byref(cov),
                                   ctypes.byref(lo), ctypes.byref(hi)), "rr_window_cover")
    return int(cov.value), int(lo.value), int(hi.value)
