"""Phase-by-phase clock trace of a decode kernel's frame loop.

    python -m paper_2510_09085_b200.phase_trace [--beam 50] [--r 1e-3] [--frames 400]
    python -m paper_2510_09085_b200.phase_trace --workload subword --beam 32     (the block kernel)
    python -m paper_2510_09085_b200.phase_trace --beam 500                       (the block kernel)

Decodes the wav2vec2-shaped batch (64 utterances, 32 tokens) with the instrumented launch of
the row kernel (``fltop_set_test_hook``, FLTOP_HOOK_PHASE_CLOCKS): every warp of utterance 0's
block records the SM clock at its phase boundaries for a range of frames.  Printed: per phase
the mean and the maximum length over the traced frames (from the moment the slowest warp left
the previous phase to the moment the slowest warp leaves this one), which warp was last, and
the same split by kind of frame.  The instrumented launch is slower than the ordinary one (a
clock read and a global store per mark), so proportions, not absolute cycle counts, are what
this is for; frames in which only blank survives have no phases and are only counted.

Vocabularies above 32 tokens and beams above 128 are decoded by the general block kernel, whose
instrumented instantiation marks its own phases (evaluate, cut, settle, write, tail); the block
traced is block 0, which in a batch of more utterances than SMs decodes the longest utterance.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as bd
from . import workloads as W

PHASES = ["evaluate (P1)", "scan (P2)", "place (P3)", "rank cut bin", "tail to next frame"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--beam", type=int, default=50)
    ap.add_argument("--r", type=float, default=1e-3)
    ap.add_argument("--first", type=int, default=50)
    ap.add_argument("--frames", type=int, default=400)
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--workload", choices=["wav2vec2", "subword"], default="wav2vec2")
    args = ap.parse_args()
    wl = W.workload_wav2vec2() if args.workload == "wav2vec2" else W.workload_subword()
    B, T, V = wl.emissions.shape
    block_kernel = V > 32 or args.beam > 128
    # (block 0 of a batch of more utterances than SMs takes the longest one)
    traced_utt = int(np.argmax(wl.lengths)) if B > 148 else 0
    nf = min(args.frames, int(wl.lengths[traced_utt]) - args.first)
    x = torch.from_numpy(wl.emissions).cuda()
    ln = torch.from_numpy(wl.lengths).cuda()
    d = bd.Decoder(V, wl.blank_id, args.beam, args.r, B, T)
    d.set_block_threads(args.threads)
    buf = torch.zeros((nf, 32, 8), dtype=torch.int64, device="cuda")
    d.decode(x, ln)
    torch.cuda.synchronize()
    d.set_test_hook(bd.FLTOP_HOOK_PHASE_CLOCKS, buf, args.first, nf)
    d.decode(x, ln)
    torch.cuda.synchronize()
    c = buf.cpu().numpy()
    if block_kernel:
        trace_block_kernel(c, args, nf)
        d.close()
        return
    nw = int((c[:, :24, 0] > 0).any(axis=0).sum())
    traced = [f for f in range(nf) if c[f, :nw, 0].min() > 0]
    print(f"K={args.beam} r={args.r:g}: {nw} warps, frames {args.first}..{args.first + nf - 1} of "
          f"utterance 0; {nf - len(traced)} of {nf} frames had only blank surviving (no phases)")
    rows, kinds, last = [], [], []
    for i, f in enumerate(traced[:-1]):
        w = c[f, :nw]
        nxt = traced[i + 1]
        if nxt != f + 1:
            continue                       # (a blank-only frame follows: no clean tail)
        start = w[:, 0].min()
        p1 = w[:, 1].max()                 # all warps have evaluated
        p2 = w[nw - 1, 3]                  # the scanning warp has published the cut
        p3 = w[:, 4].max()                 # all candidates above the cut bin are placed
        listed = w[:, 5].max() > 0
        p4 = w[:, 6].max()                 # the cut bin is ranked and written (if it had to be)
        nx = c[nxt, :nw, 0].min()
        rows.append([p1 - start, p2 - p1, p3 - p2, p4 - p3 if listed else 0, nx - (p4 if listed else p3)])
        last.append([int(w[:, 1].argmax()), nw - 1, int(w[:, 4].argmax()), int(w[:, 6].argmax()), -1])
        snb = int(c[f, 24, 5])
        kinds.append("cut bin ranked" if listed else ("many survivors (>= 16)" if snb >= 16 else "few survivors"))
    rows = np.array(rows, dtype=np.float64)
    kinds = np.array(kinds)
    last = np.array(last)
    role = lambda w: "chore" if w == nw - 1 else ("stay" if w < (args.beam + 31) // 32 else "ext")

    def show(mask, label):
        r = rows[mask]
        if not len(r):
            return
        print(f"\n{label}: {len(r)} frames, {r.sum(axis=1).mean():.0f} cycles a frame on average")
        for j, name in enumerate(PHASES):
            who = ""
            if j < 4 and (r[:, j] > 0).any():
                ws = last[mask][:, j]
                roles = [role(int(w)) for w in ws]
                who = "  last: " + ", ".join(f"{k} {roles.count(k) * 100 // len(roles)} %"
                                             for k in ("stay", "ext", "chore") if k in roles)
            print(f"  {name:20s} mean {r[:, j].mean():7.0f}  max {r[:, j].max():7.0f}{who}")
    show(np.ones(len(rows), dtype=bool), "all traced frames")
    for k in ("few survivors", "many survivors (>= 16)", "cut bin ranked"):
        show(kinds == k, k)
    d.close()


BLOCK_PHASES = ["evaluate (P1)", "cut (P2)", "settle (P3a)", "write (P3b)", "tail to next frame"]


def trace_block_kernel(c, args, nf):
    """Marks of the block kernel: 0 frame start, 1 candidates evaluated, 2 past B1, 3 cut known,
    4 candidates settled (before B3), 5 at B2 (large blocks), 6 next beam written, 7 past B4."""
    nw = int((c[:, :, 0] > 0).any(axis=0).sum())
    rows, last, skipped = [], [], 0
    for f in range(nf - 1):
        w = c[f, :nw]
        if w[:, 4].max() == 0:      # the exact select took this frame: no settle mark
            skipped += 1
            continue
        start, p1, p2 = w[:, 0].min(), w[:, 1].max(), w[:, 3].max()
        p3, p4, nx = w[:, 4].max(), w[:, 6].max(), c[f + 1, :nw, 0].min()
        rows.append([p1 - start, p2 - p1, p3 - p2, p4 - p3, nx - p4])
        last.append([int(w[:, 1].argmax()), int(w[:, 3].argmax()), int(w[:, 4].argmax()),
                     int(w[:, 6].argmax())])
    rows, last = np.array(rows, dtype=np.float64), np.array(last)
    print(f"{args.workload} K={args.beam} r={args.r:g}: block kernel, {nw} warps, frames "
          f"{args.first}..{args.first + nf - 1} of the utterance of block 0; {skipped} frames went "
          f"through the exact select (not shown)")
    print(f"\n{len(rows)} frames, {rows.sum(axis=1).mean():.0f} cycles a frame on average")
    role = lambda w: "chore" if w == nw - 1 else ("warp 0" if w == 0 else "others")
    for j, name in enumerate(BLOCK_PHASES):
        who = ""
        if j < 4:
            roles = [role(int(w)) for w in last[:, j]]
            who = "  last: " + ", ".join(f"{k} {roles.count(k) * 100 // len(roles)} %"
                                         for k in ("warp 0", "others", "chore") if k in roles)
        print(f"  {name:20s} mean {rows[:, j].mean():7.0f}  max {rows[:, j].max():7.0f}{who}")
    ok = c[: nf - 1, :nw, 4].max(axis=1) > 0
    w = c[: nf - 1, :nw][ok]
    rel = lambda mark, base: (w[:, :, mark] - base)
    s0 = w[:, :, 0].min(axis=1, keepdims=True)
    b1 = w[:, :, 2].max(axis=1, keepdims=True)
    ck = w[:, :, 3].max(axis=1, keepdims=True)
    own = w[:, :, 4] - w[:, :, 3]   # each warp's own time from knowing the cut to having settled
    print(f"  {'settled, after the warp itself knew the cut':36s} warp 0 {own[:, 0].mean():6.0f}   others mean "
          f"{own[:, 1:nw - 1].mean():6.0f} max {own[:, 1:nw - 1].max(axis=1).mean():6.0f}   chore {own[:, nw - 1].mean():6.0f}")
    for label, m, base in (("evaluated, after the frame's start", 1, s0), ("at B2, after B1", 5, b1),
                           ("settled, after the cut", 4, ck)):
        r = rel(m, base)
        print(f"  {label:36s} warp 0 {r[:, 0].mean():6.0f}   others mean {r[:, 1:nw - 1].mean():6.0f} "
              f"max {r[:, 1:nw - 1].max(axis=1).mean():6.0f}   chore {r[:, nw - 1].mean():6.0f}")


if __name__ == "__main__":
    main()
