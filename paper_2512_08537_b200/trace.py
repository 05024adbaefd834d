"""Per-item and per-pipeline-stage timeline of the head kernel (profiling aid).

    python -m paper_2512_08537_b200.trace [cfg2] [--items LO:HI]

Builds a second copy of the library with -DARDIFF_HEAD_PROFILE (libardiff_profile.so beside the regular
one; the regular library is untouched), runs the head on the survivors of the named workload and prints
what CTA 0 stamped with clock64(): for every item when the producer saw its dependencies complete and
issued its first and last copy, when the MMA issuer got its accumulator, saw the first operand slice and
issued the last MMA, when the epilogue started and finished; and for the first 16 K slices of every item
when the copy was issued and when the MMA issuer saw it complete. The profiling build is slower than the
regular one (the stamps are global stores); the timeline shows proportions, the timing comes from bench.py.
"""
from __future__ import annotations

import argparse
import ctypes
import glob
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
PROFILE_LIB = os.path.join(_HERE, "libardiff_profile.so")
TRACE_ITEMS = 4096
TYPES = ["GATHER", "COND", "IN", "SS", "GATE", "G1", "G2", "FSS", "OUT", "NOP"]


def build_profile_library() -> str:
    from . import build as lib_build
    srcs = sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cu")))
    deps = srcs + glob.glob(os.path.join(_HERE, "csrc", "*.cuh")) + [os.path.join(ROOT, "include", "ardiff.h")]
    if os.path.exists(PROFILE_LIB) and all(os.path.getmtime(p) <= os.path.getmtime(PROFILE_LIB) for p in deps):
        return PROFILE_LIB
    bdir = os.path.join(_HERE, "_build", "profile")
    os.makedirs(bdir, exist_ok=True)
    objs, procs = [], []
    for src in srcs:
        obj = os.path.join(bdir, os.path.basename(src)[:-3] + ".o")
        procs.append(subprocess.Popen([lib_build._nvcc(), *lib_build.NVCC_FLAGS, "-DARDIFF_HEAD_PROFILE", "-c", src,
                                       "-o", obj]))
        objs.append(obj)
    for p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed")
    subprocess.check_call([lib_build._nvcc(), "-shared", "-o", PROFILE_LIB, *objs, "-gencode",
                           "arch=compute_100a,code=sm_100a"])
    return PROFILE_LIB


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", nargs="?", default="cfg2")
    ap.add_argument("--items", default="60:72", help="items of CTA 0 to list one by one")
    args = ap.parse_args()
    sys.path.insert(0, ROOT)
    import torch
    import synth
    import paper_2512_08537_b200 as ardiff

    ardiff.LIB_PATH = build_profile_library()
    wl = synth.workload(args.workload)
    dev = torch.device("cuda:0")
    n = wl.n
    S = int(round(n * (1 - wl.filter_q)))
    cond = torch.from_numpy(synth.cond(wl).view(np.int16)).to(dev).view(torch.bfloat16)
    noise = torch.from_numpy(synth.noise(wl)).to(dev)
    idx = torch.randperm(n, device=dev, generator=torch.Generator(device=dev).manual_seed(1))[:S]
    idx = idx.sort().values.to(torch.int32).contiguous()
    count = torch.tensor([S], dtype=torch.int32, device=dev)
    out = torch.zeros((n, wl.C), dtype=torch.float32, device=dev)
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, n, synth.head_weights(wl))
    head.set_timing(True)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    ms, mhz = [], []
    for i in range(6):
        flush.fill_(i)
        head.ardiff_head_sample(cond, noise, synth.t_sched(wl.K), idx, count, out)
        ms.append(head.last_kernel_ms())
        mhz.append(head.last_kernel_clock_mhz())
    assert head.status() == 0
    print(f"{wl.name}: {S} survivors, K = {wl.K}; profiling build: kernel {np.median(ms[2:]):.3f} ms at "
          f"{np.median(mhz[2:]):.0f} MHz")
    raw = np.zeros(TRACE_ITEMS * 28, dtype=np.int64)
    fn = ardiff.lib().ardiff_head_copy_trace
    fn.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t]
    assert fn(head._h, raw.ctypes.data, raw.size) == 0
    tr = raw[:TRACE_ITEMS * 12].reshape(TRACE_ITEMS, 3, 4)      # [item][role: producer, MMA, epilogue][3 stamps + type]
    st = raw[TRACE_ITEMS * 12:].reshape(TRACE_ITEMS // 2, 16, 2)  # [item][K slice][issued, seen complete]
    nit = int((tr[:, 1, 2] != 0).sum())
    ty = (tr[:nit, 1, 3] // 1000).astype(int)
    period = np.diff(tr[:nit, 1, 2])
    span = tr[:nit, 1, 2] - tr[:nit, 1, 1]
    epi = tr[:nit, 2, 2] - tr[:nit, 2, 1]
    print(f"items of CTA 0: {nit}; cycles between the last MMA of consecutive items: mean {period.mean():.0f}, "
          f"median {np.median(period):.0f}")
    print(f"mean cycles: first operand slice seen -> last MMA issued {span.mean():.0f}; last MMA issued -> next "
          f"accumulator free {(tr[1:nit, 1, 0] - tr[:nit - 1, 1, 2]).mean():.0f}; accumulator free -> first slice "
          f"{(tr[1:nit, 1, 1] - tr[1:nit, 1, 0]).mean():.0f}; producer: last copy issued -> next item's "
          f"dependencies seen {(tr[1:nit, 0, 0] - tr[:nit - 1, 0, 2]).mean():.0f}")
    print("by item type:   n   MMA span   epilogue (accumulator complete -> item published)")
    for k in range(1, 9):
        sel = ty == k
        if sel.any():
            print(f"   {TYPES[k]:5s} {sel.sum():4d} {span[sel].mean():10.0f} {epi[sel].mean():10.0f}")
    lo, hi = (int(v) for v in args.items.split(":"))
    hi = min(hi, nit, TRACE_ITEMS // 2)
    lat = np.array([st[i, :, 1] - st[i, :, 0] for i in range(lo, hi) if st[i, 15, 1]])
    per = np.array([np.diff(st[i, :, 1]) for i in range(lo, hi) if st[i, 15, 1]])
    if len(lat):
        print(f"K slices of items {lo}..{hi - 1} (items with at least 16 slices):")
        print("   copy issued -> seen complete, mean per slice index:", " ".join(f"{v:.0f}" for v in lat.mean(axis=0)))
        print("   cycles between completions, mean per slice index :", " ".join(f"{v:.0f}" for v in per.mean(axis=0)))
        print(f"   overall: in flight {lat.mean():.0f} cycles, one slice completes every {per.mean():.0f} cycles")
    t0 = tr[0, 0, 0]
    print("item type.tile | producer: deps seen, first copy, last copy | MMA: accumulator free, first slice, last MMA |"
          " epilogue: deps seen, accumulator complete, published   (cycles since the first item)")
    for i in range(lo, hi):
        code = int(tr[i, 1, 3])
        print(f"{i:4d} {TYPES[code // 1000]:5s}.{code % 100:<2d} | "
              + " | ".join(" ".join(f"{int(tr[i, r, k] - t0):9d}" for k in range(3)) for r in range(3)))
    head.close()


if __name__ == "__main__":
    main()
