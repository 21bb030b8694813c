"""Timing of the separate prune kernel (Algorithm 1's conditional break over whole rows) on the
subword-shaped batch: 256 utterances, V = 1024, R = 1e-3.

    python -m paper_2510_09085_b200.prune_timing

The kernel streams the emissions once and writes the survivor lists: its algorithmic bytes are
``frames * (V * bytes per emission + 4) + survivors * 8``.  Both of its forms are timed - rows
held in registers (what a call gets) and rows staged through shared memory by asynchronous bulk
copies (``FLTOP_HOOK_PRUNE_STAGING``) - on float32 and float16 rows, with CUDA events, the L2
flushed before every launch.
"""
from __future__ import annotations

import json

import torch

from . import binding as bd
from . import workloads as W


def main():
    wl = W.workload_subword()
    B, T, V = wl.emissions.shape
    x32 = torch.from_numpy(wl.emissions).cuda()
    ln = torch.from_numpy(wl.lengths).cuda()
    frames = int(wl.lengths.sum())
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    counts = torch.zeros((B, T), dtype=torch.int32, device="cuda")
    entries = torch.zeros((B, T, V, 2), dtype=torch.int32, device="cuda")
    for dtype in (torch.float32, torch.float16):
        x = x32.to(dtype)
        for staged in (0, 1):
            d = bd.Decoder(V, 0, 32, 1e-3, B, T, emission_dtype=dtype)
            d.set_test_hook(bd.FLTOP_HOOK_PRUNE_STAGING, None, staged)
            best = None
            for i in range(10):
                flush.fill_(i)
                t0, t1 = torch.cuda.Event(True), torch.cuda.Event(True)
                t0.record()
                code = bd.fltop_prune(d.h, x, x.stride(0), x.stride(1), ln, B, T, counts, entries)
                t1.record()
                t1.synchronize()
                assert code == bd.FLTOP_OK
                if i >= 3:
                    ms = t0.elapsed_time(t1)
                    best = ms if best is None or ms < best else best
            survivors = int(counts.sum())
            nbytes = frames * (x.element_size() * V + 4) + survivors * 8
            print(json.dumps({"rows": "staged in shared memory" if staged else "in registers",
                              "emissions": str(dtype).replace("torch.", ""), "us": round(best * 1e3, 1),
                              "algorithmic_MB": round(nbytes / 1e6, 1),
                              "GB_per_s": round(nbytes / best / 1e6), "live_frames": frames,
                              "survivors": survivors}), flush=True)
            d.close()


if __name__ == "__main__":
    main()
