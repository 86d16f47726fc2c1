"""Tuning aid: where a launch of the streaming attend kernel spends its time.

Needs a library built with the phase stamps compiled in:

    LOOKAT_NVCC_FLAGS=-DLOOKAT_PHASE_STAMPS python -m paper_2601_10155_b200.build --force
    python -m paper_2601_10155_b200.phase_stamps [batch] [workload]

Prints, over the CTAs of the last of a few launches of `lookat_attend` (tables built in the kernel),
the spread of the global-timer stamps the kernel takes at its phase borders, and the spread of the
CTA durations.  The stamps are compiled out of a normal build.
"""
from __future__ import annotations

import ctypes
import sys

import numpy as np
import torch

from . import synth
from .binding import Lookat, load_library

NAMES = ["start", "first unit: barrier reached", "first unit: tables built", "first unit: tiles done",
         "last unit: tiles done", "last unit: warps merged", "end"]


def main(argv):
    batch = int(argv[1]) if len(argv) > 1 else 16
    w = synth.WORKLOADS[argv[2] if len(argv) > 2 else "gqa_32k_m8"]
    w = synth.Workload(**{**w.__dict__, "B": batch})
    lib = load_library()
    if not hasattr(lib, "lookat_debug_phase_stamps"):
        raise SystemExit("this build has no phase stamps: rebuild with LOOKAT_NVCC_FLAGS=-DLOOKAT_PHASE_STAMPS")
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    codes = torch.randint(0, w.K, (w.B, w.n_kv_heads, w.L, w.m), dtype=torch.uint8, device="cuda", generator=g)
    v = torch.randn((w.B, w.n_kv_heads, w.L, w.d_v), dtype=torch.float16, device="cuda", generator=g)
    q = torch.randn((w.B, w.n_q_heads, w.d_k), dtype=torch.float16, device="cuda", generator=g)
    books = torch.randn((w.n_kv_heads, w.m, w.K, w.d_sub), dtype=torch.float32, device="cuda", generator=g)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    out = torch.empty((w.B, w.n_q_heads, w.d_v), device="cuda")
    for _ in range(5):
        lk.lookat_attend(codes, v, q=q, codebooks=books, out=out)
    torch.cuda.synchronize()
    buf = np.zeros((1024, 8), dtype=np.uint64)
    lib.lookat_debug_phase_stamps(buf.ctypes.data_as(ctypes.c_void_p))
    used = buf[:, 6] > 0
    st = buf[used].astype(np.int64)
    rel = (st[:, :7] - st[:, 0].min()) / 1000.0
    print(f"{w.name} batch {w.B}: {used.sum()} CTAs")
    for k, name in enumerate(NAMES):
        col = rel[:, k]
        print(f"{name:30s} min {col.min():8.2f}  median {np.median(col):8.2f}  max {col.max():8.2f} us")
    dur = rel[:, 6] - rel[:, 0]
    print("CTA duration: min %.1f  p10 %.1f  median %.1f  p90 %.1f  max %.1f us"
          % (dur.min(), np.percentile(dur, 10), np.median(dur), np.percentile(dur, 90), dur.max()))
    smid = st[:, 7]
    slow = np.argsort(-dur)[:12]
    print("slowest CTAs (SM id: us):", "  ".join(f"{int(smid[i])}:{dur[i]:.0f}" for i in slow))


if __name__ == "__main__":
    main(sys.argv)
