"""Does the allocation path (and with it the page size behind the buffer) move the cliff?

    python -m paper_2405_11425_b200.alloc_study [--out DIR]

Paper, Section 1.2: the translation reach is the number of cached translations times the page
size, so a buffer mapped with larger pages should push the cliff of Section 2.1 / Fig. 1 out.
CUDA offers no page-size knob, only allocation paths that may end up with different page sizes.
This runs the unrestricted size sweep (random 128-byte lines, rr_random_read) over the same
amount of memory obtained four ways and reports the granularities the driver offers and where
the cliff falls (rr_reach) for each:

  cudaMalloc (through torch)
  virtual memory management, one physical handle, virtual address aligned to 1 GiB
  virtual memory management, one physical handle, virtual address aligned to 2 MiB
  virtual memory management, 64 MiB handles mapped side by side

Needs the cuda-python bindings (cuda.bindings.driver); nothing else in the package does.
"""
from __future__ import annotations

import argparse
import json
from pathlib import Path

from . import binding as rr

GiB = 1 << 30
SIZES_GIB = (4, 16, 32, 48, 64, 72, 80, 96, 128)


def _sweep(ptr, nbytes, nsm, out, scratch, torch):
    rr.rr_fill(ptr, nbytes // 4)
    torch.cuda.synchronize()
    pts = []
    for s in list(SIZES_GIB) + [nbytes / GiB]:
        n = int(s * GiB) // 512 * 512
        if n > nbytes or (pts and n <= pts[-1][0]):
            continue
        p = rr.ReadParams(ptr, n, W=1, warps_per_sm=32, nsm=nsm, reads_per_warp=4096, seed=7)
        rr.rr_random_read(p, out, scratch)
        g = sorted(rr.rr_random_read(p, out, scratch).gbps for _ in range(3))[1]
        pts.append((n, g))
    cliff, plateau, reach = rr.rr_reach([p[0] for p in pts], [p[1] for p in pts])
    return {"cliff": cliff, "plateau_gbps": plateau, "reach_gib": reach / GiB,
            "sweep": [[n / GiB, g] for n, g in pts]}


def run(frac_of_free: float = 0.93) -> dict:
    import torch
    from cuda.bindings import driver as drv

    def ck(r):
        if r[0] != drv.CUresult.CUDA_SUCCESS:
            raise RuntimeError(str(r[0]))
        return r[1] if len(r) == 2 else r[1:]

    torch.cuda.set_device(0)
    scratch = torch.zeros(rr.rr_scratch_bytes(), dtype=torch.uint8, device="cuda")
    info = rr.rr_device_info(scratch)
    nsm = info["nsm_prop"]
    out = torch.zeros((nsm * 32, 2), dtype=torch.int32, device="cuda")
    prop = drv.CUmemAllocationProp()
    prop.type = drv.CUmemAllocationType.CU_MEM_ALLOCATION_TYPE_PINNED
    prop.location.type = drv.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
    prop.location.id = 0
    flags = drv.CUmemAllocationGranularity_flags
    R = {"device": info["name"],
         "granularity_minimum": int(ck(drv.cuMemGetAllocationGranularity(
             prop, flags.CU_MEM_ALLOC_GRANULARITY_MINIMUM))),
         "granularity_recommended": int(ck(drv.cuMemGetAllocationGranularity(
             prop, flags.CU_MEM_ALLOC_GRANULARITY_RECOMMENDED))),
         "paths": {}}
    free, _ = torch.cuda.mem_get_info()
    size = int(free * frac_of_free) // GiB * GiB
    R["bytes"] = size

    def access(va):
        acc = drv.CUmemAccessDesc()
        acc.location.type = drv.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
        acc.location.id = 0
        acc.flags = drv.CUmemAccess_flags.CU_MEM_ACCESS_FLAGS_PROT_READWRITE
        ck(drv.cuMemSetAccess(va, size, [acc], 1))

    for align, label in ((1 << 30, "vmm one handle, address aligned to 1 GiB"),
                         (2 << 20, "vmm one handle, address aligned to 2 MiB")):
        h = ck(drv.cuMemCreate(size, prop, 0))
        va = ck(drv.cuMemAddressReserve(size, align, 0, 0))
        ck(drv.cuMemMap(va, size, 0, h, 0))
        access(va)
        try:
            R["paths"][label] = _sweep(int(va), size, nsm, out, scratch, torch)
        finally:
            torch.cuda.synchronize()
            ck(drv.cuMemUnmap(va, size))
            ck(drv.cuMemRelease(h))
            ck(drv.cuMemAddressFree(va, size))
    chunk = 64 << 20
    va = ck(drv.cuMemAddressReserve(size, 2 << 20, 0, 0))
    handles = []
    for off in range(0, size, chunk):
        h = ck(drv.cuMemCreate(chunk, prop, 0))
        ck(drv.cuMemMap(int(va) + off, chunk, 0, h, 0))
        handles.append(h)
    access(va)
    try:
        R["paths"]["vmm 64 MiB handles side by side"] = _sweep(int(va), size, nsm, out, scratch,
                                                               torch)
    finally:
        torch.cuda.synchronize()
        ck(drv.cuMemUnmap(va, size))
        for h in handles:
            ck(drv.cuMemRelease(h))
        ck(drv.cuMemAddressFree(va, size))
    t = torch.empty(size, dtype=torch.uint8, device="cuda")
    R["paths"]["cudaMalloc (torch)"] = _sweep(t, size, nsm, out, scratch, torch)
    return R


def markdown(R: dict) -> str:
    L = [f"## Allocation paths on {R['device']} ({R['bytes'] / GiB:.0f} GiB each)", "",
         f"driver granularity: minimum {R['granularity_minimum'] >> 20} MiB, recommended "
         f"{R['granularity_recommended'] >> 20} MiB", "",
         "| path | plateau GB/s | cliff | reach GiB | GB/s at " +
         " / ".join(f"{s}" for s in SIZES_GIB) + " GiB / all |", "|---|---|---|---|---|"]
    for name, r in R["paths"].items():
        L.append(f"| {name} | {r['plateau_gbps']:.0f} | {r['cliff']} | {r['reach_gib']:.0f} | "
                 + " / ".join(f"{g:.0f}" for _, g in r["sweep"]) + " |")
    return "\n".join(L) + "\n"


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="report_out")
    a = ap.parse_args(argv)
    R = run()
    out = Path(a.out)
    out.mkdir(parents=True, exist_ok=True)
    (out / "alloc_study.json").write_text(json.dumps(R, indent=1))
    (out / "alloc_study.md").write_text(markdown(R))
    print(markdown(R))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
