"""Where one pact_reduce step spends its time: start and end of every kernel on the device clock.

    python -m paper_2504_08966_b200.timeline [single_image|video|batched|stress]

Builds the instrumented copy of the library (libpact_timeline.so, -DPACT_TIMELINE: thread 0 of every CTA
stores %globaltimer when its kernel begins, each warp when it ends, and at a few points inside), replays
the step as a CUDA graph on rotating input copies and prints, per kernel, the earliest / median / latest
CTA start and end in microseconds from the start of the step.  The kernels of a step overlap through
programmatic dependent launch, so a kernel's "start" is when its CTAs were scheduled, not when its
predecessor finished; the step time printed by bench.py is taken with the uninstrumented library.
"""
from __future__ import annotations

import ctypes as C
import sys

import numpy as np
import torch

from . import binding as pb
from . import build as pact_build
from . import workloads

KERNELS = {0: "k_qsum", 1: "k_tokens", 2: "k_scores", 3: "k_select", 4: "k_tiles_umma<gram>", 5: "k_centers",
           6: "k_tiles_umma<assign>", 7: "  k_select: threshold known", 8: "k_members / k_lists", 9: "k_merge",
           10: "  k_centers: keys staged", 11: "  k_centers: sweeps done", 12: "  k_centers: after grid barrier",
           13: "  members: labels read", 14: "  members: offsets known", 15: "  k_merge: records read"}
SLOTS, CTAS = 16, 4096


def main(name: str = "single_image") -> None:
    pb.LIB_PATH = pact_build.build(timeline=True)
    L = pb.lib()
    buf = torch.zeros(SLOTS * CTAS * 2, dtype=torch.int64, device="cuda")
    L.pact_debug_set_timeline.argtypes = [C.c_void_p]
    L.pact_debug_set_timeline.restype = None
    L.pact_debug_set_timeline(C.c_void_p(buf.data_ptr()))
    wl = workloads.build(name, seed={"single_image": 1, "video": 3, "batched": 2, "stress": 4}[name])
    params = pb.make_params(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha)
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.bfloat16)
    sets = [[pb.device_image(img, torch.bfloat16) for img in wl.images] for _ in range(3)]
    graphs = [ctx.pact_graph_create(ims, params) for ims in sets]
    for i in range(12):
        graphs[i % 3].launch()
    torch.cuda.synchronize()
    buf.zero_()
    torch.cuda.synchronize()
    graphs[0].launch()
    torch.cuda.synchronize()
    a = buf.cpu().numpy().reshape(SLOTS, CTAS, 2)
    t0 = a[a > 0].min()
    print(f"{wl.name}: one graph replay, first image of the batch; microseconds from the first CTA start")
    print(f"{'kernel / point':34s} {'CTAs':>5s}   start min / median / max      end min / median / max")
    for k in range(SLOTS):
        s, e = a[k, :, 0], a[k, :, 1]
        m = s > 0
        if not m.any():
            continue
        s, e = (s[m] - t0) / 1e3, (e[m] - t0) / 1e3
        line = f"{KERNELS.get(k, str(k)):34s} {int(m.sum()):5d}   {s.min():7.2f} {np.median(s):7.2f} {s.max():7.2f}"
        if not KERNELS.get(k, "").startswith("  "):
            line += f"   {e.min():7.2f} {np.median(e):7.2f} {e.max():7.2f}"
        print(line)


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else "single_image")
