"""Comparison protocol between the CUDA library and the CPU oracle.

Survivor sets are compared bit for bit.  Hypotheses are matched by token
sequence: the top-1 sequences must be identical unless the oracle's two best
scores are closer than the tolerance; matched scores must agree within the
tolerance (1e-3 nats absolute); a CUDA hypothesis the oracle does not list is
accepted only next to the cut, i.e. when its score is within the tolerance of
the oracle's last kept score (float32 vs float64 rounding can swap two
candidates that are that close).  The number of such swaps is returned.
"""
from __future__ import annotations

import numpy as np

TOL = 1e-3


def check_hyps(gpu, ora, K, tol=TOL, max_unmatched_frac=0.0, where=""):
    """gpu / ora: [(token tuple, score)], best first.  Returns #unmatched."""
    assert len(gpu) == len(ora), f"{where}: {len(gpu)} hypotheses vs oracle {len(ora)}"
    if not ora:
        return 0
    assert len(set(s for s, _ in gpu)) == len(gpu), f"{where}: duplicate prefixes in the beam"
    top_gap = ora[0][1] - ora[1][1] if len(ora) > 1 else np.inf
    if gpu[0][0] != ora[0][0]:
        assert top_gap < tol, f"{where}: top-1 differs with oracle gap {top_gap}"
    omap = dict(ora)
    cut = ora[-1][1]
    unmatched = 0
    for seq, sc in gpu:
        if seq in omap:
            assert abs(sc - omap[seq]) <= tol, \
                f"{where}: score {sc} vs oracle {omap[seq]} for a {len(seq)}-token hypothesis"
        else:
            unmatched += 1
            if max_unmatched_frac == 0.0:
                assert len(ora) == K and sc <= cut + tol, \
                    f"{where}: hypothesis not in the oracle beam, score {sc}, cut {cut}"
    assert unmatched <= max(1, int(max_unmatched_frac * len(ora))) or max_unmatched_frac == 0.0, \
        f"{where}: {unmatched} of {len(ora)} hypotheses unmatched"
    sc = [s for _, s in gpu]
    assert all(sc[i] >= sc[i + 1] for i in range(len(sc) - 1)), f"{where}: not sorted best first"
    return unmatched


def masks_from_entries(counts, entries, V):
    """counts [B,T] int32, entries [B,T,V,2] int32 -> keep [B,T,V] bool, logp [B,T,V] f32 (nan = pruned)."""
    B, T = counts.shape
    keep = np.zeros((B, T, V), dtype=bool)
    vals = np.full((B, T, V), np.nan, dtype=np.float32)
    tok = entries[..., 0]
    lp = entries[..., 1].view(np.float32)
    for b in range(B):
        for t in range(T):
            n = counts[b, t]
            if n:
                tk = tok[b, t, :n]
                assert (np.diff(tk) > 0).all(), "survivors not in ascending token order"
                keep[b, t, tk] = True
                vals[b, t, tk] = lp[b, t, :n]
    return keep, vals
