"""Comparison protocol between the CUDA library and the CPU oracle.

Survivor sets are compared bit for bit.  Hypotheses are matched by token
sequence: the top-1 sequences must be identical unless the oracle's two best
scores are closer than the tolerance; matched scores must agree within the
tolerance (1e-3 nats absolute).

Where float32 and float64 arithmetic rank two candidates of a frame differently
(a near-tie at the cut), the two beams can end with different tails, and several
results are correct.  A CUDA hypothesis that the oracle's beam does not hold is
therefore not compared with the oracle but checked for validity on its own:

* its score may not exceed the exact log-probability of its token sequence on the
  pruned frames - the CTC forward recursion over all alignments, computed here in
  float64 (``tests/refs.py``), of which every beam-search score is a lower bound;
* its score may not lie below the oracle's last kept score by more than
  ``CASCADE`` (a swap at the cut exchanges two candidates of nearly equal score,
  so what the swapped-in prefix grows into ends next to the cut as well).  Inputs
  on which scores tie exactly all the time (emissions rounded to bfloat16, flat
  rows) pass a wider ``cascade``: there the two sides may break a tie differently
  many frames before the end.

A hypothesis within the tolerance of the oracle's last kept score is a swap at the final
cut and always acceptable.  Of the others callers state how many they tolerate (none on
small cases and on the benchmark batch).  The number of unmatched hypotheses is returned.
"""
from __future__ import annotations

import numpy as np

from tests.refs import ctc_forward_logprob

TOL = 1e-3
CASCADE = 10 * TOL


def check_hyps(gpu, ora, K, tol=TOL, max_unmatched_frac=0.0, where="", lp=None, keep=None,
               blank=0, cascade=CASCADE):
    """gpu / ora: [(token tuple, score)], best first.  Returns the number of CUDA hypotheses
    that the oracle's beam does not hold.

    ``lp`` [T,V] (and ``keep`` [T,V], the frame-level survivor masks) are the utterance's
    emissions: with them every unmatched hypothesis is checked against the exact CTC forward
    probability of its sequence.  Without them unmatched hypotheses are accepted only next
    to the oracle's cut."""
    assert len(gpu) == len(ora), f"{where}: {len(gpu)} hypotheses vs oracle {len(ora)}"
    if not ora:
        return 0
    assert len(set(s for s, _ in gpu)) == len(gpu), f"{where}: duplicate prefixes in the beam"
    top_gap = ora[0][1] - ora[1][1] if len(ora) > 1 else np.inf
    if gpu[0][0] != ora[0][0]:
        assert top_gap < tol, f"{where}: top-1 differs with oracle gap {top_gap}"
    omap = dict(ora)
    cut = ora[-1][1]
    at_cut = beyond = 0
    for seq, sc in gpu:
        if seq in omap:
            assert abs(sc - omap[seq]) <= tol, \
                f"{where}: score {sc} vs oracle {omap[seq]} for a {len(seq)}-token hypothesis"
            continue
        # a full oracle beam is the only way a correct hypothesis can be missing from it
        assert len(ora) == K, f"{where}: hypothesis missing from an oracle beam that is not full"
        assert sc >= cut - cascade, \
            f"{where}: unmatched hypothesis scores {sc}, far below the oracle's cut {cut}"
        if lp is not None:
            exact = ctc_forward_logprob(lp, seq, blank, keep)
            assert sc <= exact + tol, \
                f"{where}: unmatched hypothesis scores {sc} above its exact probability {exact}"
        if sc <= cut + tol:
            at_cut += 1      # swapped with an oracle hypothesis of (nearly) the same score
        else:
            assert lp is not None, \
                f"{where}: hypothesis not in the oracle beam, score {sc}, cut {cut}"
            beyond += 1      # grown from a swap at the cut of an earlier frame
    allowed = int(max_unmatched_frac * len(ora))
    assert beyond <= allowed, \
        f"{where}: {beyond} of {len(ora)} hypotheses not in the oracle beam (allowed {allowed})"
    sc = [s for _, s in gpu]
    assert all(sc[i] >= sc[i + 1] for i in range(len(sc) - 1)), f"{where}: not sorted best first"
    return at_cut + beyond


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


def masks_from_words(words, V):
    """words [..] uint32 survivor masks (bit c = token c) -> keep [.., V] bool."""
    w = np.asarray(words).astype(np.uint32)
    return ((w[..., None] >> np.arange(V, dtype=np.uint32)) & 1).astype(bool)
