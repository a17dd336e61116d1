"""Per-phase timeline of the fused attention kernel, from clock64() stamps of one CTA.

Developer tool.  The stamps exist only in a library built with the trace switch::

    BAPS_NVCC_EXTRA=-DBAPS_TRACE=1 python -m paper_2602_02071_b200.build --force
    python -m paper_2602_02071_b200.timeline            # long causal case, B1 H8 Hkv2 S16384 D128
    python -m paper_2602_02071_b200.build --force       # back to the normal build

It prints, for the steady state of CTA 0 (the heaviest one), the mean number of cycles per task and
per phase of the softmax warps, the spread between the sixteen warps, and the timing of the MMA
warp's burst.  Numbers taken with the switch on are a little slower than the normal build (every
stamp is a clock read and a global store) and are never benchmark values.
"""
from __future__ import annotations

import ctypes
import sys

import numpy as np
import torch

from . import binding, workloads

SLOTS, MMA_SLOTS, MAX_TASKS = 8, 8, 600


def main(seq: int = 16384) -> int:
    lib = binding.load()
    if not hasattr(lib, "baps_debug_trace_read"):
        print("this library was built without -DBAPS_TRACE=1", file=sys.stderr)
        return 1
    w = workloads.AttnWorkload("timeline", 1, 8, 2, seq, 128, True, 128, 128)
    q, k, v = workloads.make_qkv(w, device="cuda")
    for _ in range(2):
        binding.baps_attention_fwd(q, k, v, causal=True)
    torch.cuda.synchronize()
    buf = np.zeros(MAX_TASKS * 16 * SLOTS, dtype=np.int64)
    mbuf = np.zeros(MAX_TASKS * MMA_SLOTS, dtype=np.int64)
    lib.baps_debug_trace_read.argtypes = [ctypes.c_void_p]
    lib.baps_debug_trace_read_mma.argtypes = [ctypes.c_void_p]
    assert lib.baps_debug_trace_read(buf.ctypes.data) == 0
    assert lib.baps_debug_trace_read_mma(mbuf.ctypes.data) == 0
    ntasks = min(MAX_TASKS, 4 * (seq // 256 - 1) + 3)
    lo, hi = 20, ntasks - 15                               # steady state of CTA 0
    tr = buf.reshape(MAX_TASKS, 16, SLOTS)[lo:hi]
    mm = mbuf.reshape(MAX_TASKS, MMA_SLOTS)[lo:hi]
    print(f"tasks {lo}..{hi} of {ntasks}: {np.diff(tr[:, 0, 0]).mean():.0f} cycles per task")
    for name, a, b in (("start -> scores in registers", 0, 1), ("-> maxima exchanged, verdict", 1, 2),
                       ("-> weights done", 2, 3), ("-> P stored, arrived", 3, 5), ("-> next scores requested", 5, 4)):
        dt = tr[:, :, b] - tr[:, :, a]
        print(f"  {name:32s} mean {dt.mean():6.0f}   (slowest warp {dt.mean(0).max():.0f}, fastest {dt.mean(0).min():.0f})")
    print(f"  -> next task start               mean {(tr[1:, :, 0] - tr[:-1, :, 4]).mean():6.0f}")
    wph = tr[:, :, 3] - tr[:, :, 2]
    print("  weights phase over warps and tasks: p10 %.0f  p50 %.0f  p90 %.0f" % tuple(np.percentile(wph, [10, 50, 90])))
    print(f"  skew between warps: at task start {(tr[:, :, 0].max(1) - tr[:, :, 0].min(1)).mean():.0f}, "
          f"at arrival {(tr[:, :, 5].max(1) - tr[:, :, 5].min(1)).mean():.0f}")
    last_arrive = tr[:, :, 5].max(1)
    print(f"MMA warp: last arrival -> P seen {(mm[:, 1] - last_arrive).mean():.0f}; P seen -> first MMA "
          f"{(mm[:, 5] - mm[:, 1]).mean():.0f}; 16 MMAs issued in {(mm[:, 6] - mm[:, 5]).mean():.0f}; "
          f"commits {(mm[:, 7] - mm[:, 6]).mean():.0f}; waits for K/V before P {(mm[:, 3] - mm[:, 0]).mean():.0f}")
    return 0


if __name__ == "__main__":
    sys.exit(main(int(sys.argv[1]) if len(sys.argv) > 1 else 16384))
