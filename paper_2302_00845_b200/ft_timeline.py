"""Phase timeline of the TMA-fed FMA pass 1 (m <= 16, long rows), from the stamp build.

    python -m paper_2302_00845_b200.ft_timeline [--d D] [--m M] [--dtype f32|bf16] [--steps K]

Builds libcdgrab_stamp.so (-DCDGRAB_STAMP: every CTA records %globaltimer at its phase
boundaries), runs K steps of the mid-size recipe on two alternating buffers and prints, for the
last launch, min / median / max over the CTAs of each boundary in microseconds after the first
CTA passed the dependency wait.  Set CDGRAB_FT_WHOLE=1 to see the single-launch form.
"""
from __future__ import annotations

import argparse
import ctypes as C
import os
import sys

os.environ["CDGRAB_LIB"] = "libcdgrab_stamp.so"      # before the binding is imported

import numpy as np  # noqa: E402
import torch  # noqa: E402

from . import binding, build, synth  # noqa: E402

SLOTS = 16
NAMES = [(0, "barriers ready"), (1, "dependency wait over"), (2, "first tile landed"), (3, "pass 1 loop done"),
         (4, "ticket taken"), (5, "all groups finished (wait over)"), (12, "totals visible"),
         (13, "group partials summed"), (14, "decisions taken"), (6, "signs in shared memory"),
         (7, "pass 2: ring tiles done"), (8, "pass 2: first reloaded tile landed"), (9, "pass 2 done")]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d", type=int, default=1 << 20)
    ap.add_argument("--m", type=int, default=16)
    ap.add_argument("--dtype", default="f32")
    ap.add_argument("--steps", type=int, default=12)
    a = ap.parse_args()
    build.build(variant="stamp")
    wl = synth.WORKLOADS["mid"].scaled(m=a.m, n=2 * a.steps, d=a.d, dtype=a.dtype)
    gs = synth.GradientStream(wl, device="cuda")
    bufs = [gs.step(k) for k in range(2)]
    lib = binding.lib()
    lib.cdgrab_debug_ft_stamps.argtypes = [C.c_void_p, C.c_int]
    with binding.CdGrab(wl.m, wl.n, wl.d, wl.dtype) as h:
        assert h.path == "fma"
        h.begin_epoch()
        for k in range(a.steps):
            h.step(bufs[k & 1])
        ctas = min(torch.cuda.get_device_properties(0).multi_processor_count, (a.d + 255) // 256)
        out = np.zeros((ctas, SLOTS), dtype=np.uint64)
        assert lib.cdgrab_debug_ft_stamps(out.ctypes.data, ctas) == 0
        h.check_status()
    t = out.astype(np.int64)
    t0 = t[:, 1].min()
    print(f"m={wl.m} d={wl.d} {wl.dtype}, {ctas} CTAs; launch gap (first entry - last exit of the launch before, "
          f"single-launch form only): {(t[:, 10].min() - t[:, 11].max()) / 1e3:.2f} us")
    for slot, name in NAMES:
        col = (t[:, slot] - t0) / 1e3
        col = col[t[:, slot] >= t[:, 10]]        # stamped during the last launch (not a leftover of an earlier one)
        if col.size:
            print(f"{name:38s} min {col.min():8.2f}  median {np.median(col):8.2f}  max {col.max():8.2f} us"
                  f"   ({col.size} CTAs)")


if __name__ == "__main__":
    main()
